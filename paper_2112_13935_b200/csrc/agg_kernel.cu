// Server side: ordered aggregation of the triggered update sums.
//
// Algorithm 3, Receive: "w = w - eta_k * U; H_v = H_v + 1", applied in the
// order the simulated-time schedule fixes.  Each thread owns a few parameters
// and walks the updates of the range in order, keeping its parameters in
// registers; wherever a later round starts from the model after update k the
// running value is also stored as that round's start snapshot (this replaces a
// separate broadcast copy into client slots).  The walk is sequential in k, as
// the paper's server is, and parallel over parameters.
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "aet_kernels.h"

namespace aet {
namespace {

constexpr int kAggThreads = 128;
constexpr int kAhead = 8;  // update rows fetched ahead of the dependent FMA chain

__global__ void __launch_bounds__(kAggThreads) apply_updates_kernel(ApplyLaunch p) {
  const uint32_t j = blockIdx.x * kAggThreads + threadIdx.x;
  if (j < p.n_params) {
    float w = p.w_cur[j];
    const float* U = p.U + j;
    uint32_t k = p.lo;
    for (; k + kAhead <= p.hi; k += kAhead) {
      float u[kAhead];
#pragma unroll
      for (int a = 0; a < kAhead; ++a) u[a] = __ldcs(U + (size_t)(k + a) * p.stride);
#pragma unroll
      for (int a = 0; a < kAhead; ++a) {
        const ApplyDesc d = p.applies[k + a];
        w = fmaf(-d.eta, u[a], w);
        if (d.snap_slot >= 0) p.snaps[(size_t)d.snap_slot * p.stride + j] = w;
      }
    }
    for (; k < p.hi; ++k) {
      const ApplyDesc d = p.applies[k];
      w = fmaf(-d.eta, __ldcs(U + (size_t)k * p.stride), w);
      if (d.snap_slot >= 0) p.snaps[(size_t)d.snap_slot * p.stride + j] = w;
    }
    p.w_cur[j] = w;
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    for (uint32_t k = p.lo; k < p.hi; ++k) {
      const ApplyDesc d = p.applies[k];
      ApplyRec r;
      r.client = d.client; r.round = d.round; r.seq = k;
      r.h_after = ++p.H[d.client];
      p.log[k] = r;
    }
  }
}

__global__ void to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t step = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += step) dst[i] = __float2bfloat16_rn(src[i]);
}

}  // namespace

cudaError_t launch_apply_updates(const ApplyLaunch& p, cudaStream_t s) {
  if (p.hi <= p.lo) return cudaSuccess;
  const uint32_t blocks = (p.n_params + kAggThreads - 1) / kAggThreads;
  apply_updates_kernel<<<blocks, kAggThreads, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_to_bf16(const float* src, void* dst, size_t n, cudaStream_t s) {
  if (!n) return cudaSuccess;
  size_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  to_bf16_kernel<<<(unsigned)blocks, 256, 0, s>>>(src, reinterpret_cast<__nv_bfloat16*>(dst), n);
  return cudaGetLastError();
}

}  // namespace aet
