// Pieces shared by the MLP round kernels: cluster helpers and the layout of the
// per-task global scratch (partial products, dZ and activations of every layer).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "aet_kernels.h"

namespace aet {
namespace mlp {

__device__ __forceinline__ void cluster_sync(bool clustered) {
  if (clustered) {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  } else {
    __threadfence_block();
    __syncthreads();
  }
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ float q_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
__device__ __forceinline__ int up4(int v) { return (v + 3) & ~3; }

struct Layout {  // offsets (in floats) into the per-task global scratch
  size_t part[AET_MAX_LAYERS], dz[AET_MAX_LAYERS], a[AET_MAX_LAYERS], total;
};
__host__ __device__ inline Layout make_layout(const MlpShape& s) {
  Layout L{};
  size_t o = 0;
  for (uint32_t l = 0; l < s.n_layers; ++l) {
    const size_t bn = (size_t)s.batch * s.dims[l + 1];
    L.part[l] = o; o += (size_t)s.cluster * bn;
    L.dz[l] = o; o += bn;
    L.a[l] = o; o += bn;
  }
  L.total = (o + 31) & ~(size_t)31;
  return L;
}

// Element-wise copy with kInFlight loads in flight per thread before the first
// store (the compiler cannot reorder global loads across shared-memory stores
// itself, and a dependent round trip to L2 costs about a microsecond).
constexpr int kInFlight = 8;
template <int kThreadsT, class Load, class Store>
__device__ __forceinline__ void staged_copy_t(int total, int tid, Load ld, Store st) {
  for (int e0 = tid; e0 < total; e0 += kInFlight * kThreadsT) {
    float v[kInFlight];
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) { const int e = e0 + u * kThreadsT; v[u] = e < total ? ld(e) : 0.f; }
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) { const int e = e0 + u * kThreadsT; if (e < total) st(e, v[u]); }
  }
}

}  // namespace mlp
}  // namespace aet
