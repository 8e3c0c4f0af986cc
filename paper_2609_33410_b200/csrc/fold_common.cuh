// Shared device helpers for the fold decode kernels (sm_100a): mbarrier / TMA / ldmatrix /
// mma.sync / cp.async wrappers, the canonical chunk rule and small numeric helpers.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "fold.h"

namespace fold {

constexpr int kTileKeys = 64;            // keys per tile (Algorithm 1 walks 64-key tiles)
// Narrow row blocks walk 16 KB key tiles whatever the head dimension (64 keys at D = 128, 128 at D = 64), so a
// warp's slice is always 4 KB of keys and the per-slice costs (waits, hand-offs) are paid per byte alike.
constexpr int kNarrowRows = 8;           // row blocks up to this size put the rows on the MMA's N side
template <int D>
__host__ __device__ constexpr int narrow_tile_keys() { return 8192 / D; }
constexpr int kConsumerWarps = 4;        // each owns 16 keys of every tile
constexpr int kScanThreads = (kConsumerWarps + 1) * 32;   // + one producer warp
constexpr int kMaxRows = 16;             // query rows one row block holds (MMA M)
constexpr int kMaxLevels = 4;
constexpr uint32_t kWaitLimit = 1u << 20;   // bounded spins: give up, flag, fall through

// Canonical chunk rule.  A function of the sequence's own length only, so that a slot's
// content cannot depend on the batch it is decoded in or on the split count.
__host__ __device__ inline int chunk_keys_of(int n) { return n <= 8192 ? 256 : 1024; }
__host__ __device__ inline int num_chunks_of(int n) {
  const int c = chunk_keys_of(n);
  return (n + c - 1) / c;
}
// Largest chunk count any sequence of at most n keys can have.
__host__ __device__ inline int max_chunks_upto(int n) {
  if (n <= 8192) return (n + 255) / 256;
  const int a = (n + 1023) / 1024;
  return a > 32 ? a : 32;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- programmatic dependent launch
// A kernel launched with the programmatic-serialization attribute may start while the kernel
// before it in the stream is still running; it must not touch that kernel's results before
// pdl_wait().  pdl_launch_dependents() lets the next kernel's CTAs be scheduled early.  Both are
// no-ops when the launch carries no such attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {   // no arrival: bytes only
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the phase never completed within the limit; `dead`
// short-circuits every later wait of a thread that has already given up once.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, bool &dead) {
  if (dead) return false;
  for (uint32_t i = 0; i < kWaitLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  dead = true;
  return false;
}
// The same with a non-suspending probe: a thread on a latency-critical hand-off polls instead of sleeping.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_spin(uint32_t bar, uint32_t parity, bool &dead) {
  if (dead) return false;
  for (uint32_t i = 0; i < 16u * kWaitLimit; ++i)
    if (mbar_test_wait(bar, parity)) return true;
  dead = true;
  return false;
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- TMA (no multicast)
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
// Plain (untiled) bulk copy global -> shared of `bytes` (multiple of 16; both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// The same box fetched into L2 only: no shared memory, no completion to wait for.
__device__ __forceinline__ void tma_prefetch_l2_4d(const CUtensorMap *map, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// ---------------------------------------------------------------- cp.async (16-byte, zero-fill when src_bytes == 0)
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// Ties the completion of this thread's earlier cp.async copies to an mbarrier phase: the pending count
// goes up by one now and down by one when those copies have landed.
__device__ __forceinline__ void cp_async_mbar_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ---------------------------------------------------------------- ldmatrix / mma.sync (BF16 in, FP32 accumulate)
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ---------------------------------------------------------------- numerics
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Two-term BF16 split of a weight (Algorithm 1: P_hi = bf16(p), P_lo = bf16(p - P_hi)).
__device__ __forceinline__ void split_bf16(float p, float &hi, float &lo) {
  hi = __bfloat162float(__float2bfloat16_rn(p));
  lo = __bfloat162float(__float2bfloat16_rn(p - hi));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo_elem, float hi_elem) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo_elem, hi_elem);   // .x (low 16 bits) = lo_elem
  return *reinterpret_cast<uint32_t *>(&v);
}

// Byte offset of the 16-byte chunk `c16` (0 .. D/8-1) of token row `tok` inside a tile laid
// out as [D/64 halves][tokens][128 bytes] with the 128-byte TMA swizzle (chunk index XOR
// row index mod 8).  `rows` = token rows per half.
__device__ __forceinline__ uint32_t tile_off(int tok, int c16, int rows) {
  return static_cast<uint32_t>(((c16 >> 3) * rows + tok) * 128 + (((c16 & 7) ^ (tok & 7)) << 4));
}

}  // namespace fold
