// Read-only bandwidth probe: streams a buffer once with 16-byte loads on every SM and folds what it read into one
// word, so nothing is optimised away.  It gives the scans' roofline its third denominator: the measured copy figure
// counts read + write traffic, the nominal figure is a data-sheet number, this is what a kernel that only reads
// actually gets from this memory system.
#pragma once

#include "fold_common.cuh"

namespace fold {

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;

__global__ void __launch_bounds__(kProbeThreads) fold_probe_read_kernel(const uint4 *__restrict__ src, size_t n16,
                                                                         unsigned long long *sink) {
  const size_t stride = (size_t)gridDim.x * kProbeThreads;
  size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
  uint32_t acc = 0;
  for (; i + (kProbeUnroll - 1) * stride < n16; i += kProbeUnroll * stride) {
    uint4 v[kProbeUnroll];
#pragma unroll
    for (int u = 0; u < kProbeUnroll; ++u)                    // streaming loads: read once, evict first
      asm volatile("ld.global.cs.v4.u32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                   : "l"(src + i + u * stride));
#pragma unroll
    for (int u = 0; u < kProbeUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = src[i];
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  acc = __reduce_xor_sync(0xffffffffu, acc);
  if ((threadIdx.x & 31) == 0 && sink) atomicXor(sink, (unsigned long long)acc);
}

}  // namespace fold
