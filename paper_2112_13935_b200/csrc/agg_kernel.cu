// Server side: ordered aggregation of the triggered update sums.
//
// Algorithm 3, Receive: "w = w - eta_k * U; H_v = H_v + 1", applied in the
// order the simulated-time schedule fixes.  Each thread owns one parameter and
// walks the updates of its range in order, keeping the parameter in a register;
// wherever a later round starts from the model after update k the running
// value is also stored as that round's start snapshot (this replaces a
// separate broadcast copy into client slots).
//
// A long range (many clients) is cut into G groups of consecutive updates.
// Pass 1 sums -eta_k * U_k over each group; pass 2 starts group g from
// w + sum of the totals of the groups before it and walks the group in order.
// The result is the paper's sequential rule up to fp32 re-association across
// group boundaries, and identical from run to run.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "aet_kernels.h"

namespace aet {
namespace {

constexpr int kAggThreads = 128;
constexpr int kAhead = 8;  // update rows fetched ahead of the dependent FMA chain

__device__ __forceinline__ void group_range(const ApplyLaunch& p, uint32_t g, uint32_t& lo, uint32_t& hi) {
  const uint32_t per = (p.hi - p.lo + p.groups - 1) / p.groups;
  lo = min(p.hi, p.lo + g * per);
  hi = min(p.hi, lo + per);
}

// Both kernels are launched with programmatic stream serialisation: their CTAs may become resident
// while the kernel ahead of them in the stream (the round kernel, then group_totals_kernel) is
// draining, and they read and write nothing before griddepcontrol.wait, which returns once that
// kernel - and, because it waited the same way, every kernel before it - has finished.
__global__ void __launch_bounds__(kAggThreads) group_totals_kernel(ApplyLaunch p) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t j = blockIdx.x * kAggThreads + threadIdx.x;
  if (j >= p.n_params) return;
  uint32_t lo, hi;
  group_range(p, blockIdx.y, lo, hi);
  const float* U = p.U + j;
  float s = 0.f;
  uint32_t k = lo;
  for (; k + kAhead <= hi; k += kAhead) {
    float u[kAhead];
#pragma unroll
    for (int a = 0; a < kAhead; ++a) u[a] = __ldg(U + (size_t)p.applies[k + a].u_row * p.stride);
#pragma unroll
    for (int a = 0; a < kAhead; ++a) s = fmaf(-p.applies[k + a].eta, u[a], s);
  }
  for (; k < hi; ++k) s = fmaf(-p.applies[k].eta, __ldg(U + (size_t)p.applies[k].u_row * p.stride), s);
  p.totals[(size_t)blockIdx.y * p.stride + j] = s;
}

__global__ void __launch_bounds__(kAggThreads) apply_updates_kernel(ApplyLaunch p) {
  // The round kernel that follows in the stream may be launched with programmatic stream
  // serialisation: let its CTAs start their set-up (descriptors, first rows) while this grid
  // runs.  They read nothing this grid writes before their own griddepcontrol.wait, which
  // returns only once this grid has finished and its writes are visible.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const uint32_t j = blockIdx.x * kAggThreads + threadIdx.x;
  const uint32_t g = blockIdx.y;
  uint32_t lo, hi;
  group_range(p, g, lo, hi);
  if (j < p.n_params) {
    float w = p.w_in[j];
    for (uint32_t q = 0; q < g; ++q) w += p.totals[(size_t)q * p.stride + j];
    const float* U = p.U + j;
    uint32_t k = lo;
    for (; k + kAhead <= hi; k += kAhead) {
      float u[kAhead];
#pragma unroll
      ApplyDesc ds[kAhead];
#pragma unroll
      for (int a = 0; a < kAhead; ++a) ds[a] = p.applies[k + a];
#pragma unroll
      for (int a = 0; a < kAhead; ++a) u[a] = __ldcs(U + (size_t)ds[a].u_row * p.stride);
#pragma unroll
      for (int a = 0; a < kAhead; ++a) {
        const ApplyDesc d = ds[a];
        w = fmaf(-d.eta, u[a], w);
        if (d.snap_slot >= 0) p.snaps[(size_t)d.snap_slot * p.stride + j] = w;
      }
    }
    for (; k < hi; ++k) {
      const ApplyDesc d = p.applies[k];
      w = fmaf(-d.eta, __ldcs(U + (size_t)d.u_row * p.stride), w);
      if (d.snap_slot >= 0) p.snaps[(size_t)d.snap_slot * p.stride + j] = w;
    }
    if (g + 1 == p.groups) {
      p.w_out[j] = w;
      // the server model after this range: a non-finite entry (a NaN or an overflow that came in
      // through a client's rows or step size) is reported, never trapped on
      if (p.status && !isfinite(w)) atomicOr(p.status, 2u);
    }
  }
  // history map and apply log: one thread per update of the group
  if (blockIdx.x == 0)
    for (uint32_t k = lo + threadIdx.x; k < hi; k += kAggThreads) {
      const ApplyDesc d = p.applies[k];
      ApplyRec r;
      r.client = d.client; r.round = d.round; r.seq = k;
      r.h_after = atomicAdd(&p.H[d.client], 1u) + 1u;
      p.log[k] = r;
    }
}

__global__ void to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t step = (size_t)gridDim.x * blockDim.x;
  for (; i < n; i += step) dst[i] = __float2bfloat16_rn(src[i]);
}

// Peer-to-peer ring: Receive at every node (Algorithm 3: w_c = w_c - eta_k * U) for the sums that
// reached it, preceded by the node's own sum of the round it has just finished.  One y-block per node
// whose model moves; a thread keeps its parameter in a register and walks the node's short list.
__global__ void __launch_bounds__(kAggThreads) ring_apply_kernel(RingApplyLaunch p) {
  const uint32_t j = blockIdx.x * kAggThreads + threadIdx.x;
  if (j >= p.n_params) return;
  const RingApplyDesc a = p.applies[p.lo + blockIdx.y];
  float* wp = p.node_w + (size_t)a.node * p.stride + j;
  float w = *wp;
  for (uint32_t k = 0; k < a.op_cnt; ++k) {
    const RingOp op = p.ops[a.op_off + k];
    w = fmaf(-op.eta, __ldg(p.U + (size_t)op.u_row * p.stride + j), w);
  }
  *wp = w;
  if (p.status && !isfinite(w)) atomicOr(p.status, 2u);
}

// Debug pass over a client's data set as it is loaded: a label outside [0, n_classes) sets bit 2
// of *status, a non-finite pixel bit 1.  Nothing is trapped on; the host turns the bits into
// AET_ERR_STATE / AET_ERR_NUMERIC at its next synchronising call.
__global__ void validate_data_kernel(const float* __restrict__ x, const int32_t* __restrict__ y, uint32_t n,
                                     uint32_t dim, uint32_t n_classes, uint32_t* status) {
  const size_t step = (size_t)gridDim.x * blockDim.x;
  uint32_t bad = 0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += step)
    if ((uint32_t)y[i] >= n_classes) bad |= 4u;
  if (x)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)n * dim; i += step)
      if (!isfinite(x[i])) bad |= 2u;
  if (bad) atomicOr(status, bad);
}

}  // namespace

cudaError_t launch_validate_data(const float* x, const int32_t* y, uint32_t n, uint32_t dim, uint32_t n_classes,
                                 uint32_t* status, cudaStream_t s) {
  if (!n) return cudaSuccess;
  size_t blocks = ((size_t)n * dim + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  validate_data_kernel<<<(unsigned)blocks, 256, 0, s>>>(x, y, n, dim, n_classes, status);
  return cudaGetLastError();
}

cudaError_t launch_ring_apply(const RingApplyLaunch& p, cudaStream_t s) {
  if (p.hi <= p.lo) return cudaSuccess;
  const uint32_t blocks = (p.n_params + kAggThreads - 1) / kAggThreads;
  ring_apply_kernel<<<dim3(blocks, p.hi - p.lo, 1), kAggThreads, 0, s>>>(p);
  return cudaGetLastError();
}

uint32_t apply_groups(uint32_t n_updates) {
  uint32_t g = n_updates / 32;
  return g < 1 ? 1 : (g > 32 ? 32 : g);
}

cudaError_t launch_apply_updates(const ApplyLaunch& p, cudaStream_t s) {
  if (p.hi <= p.lo) return cudaSuccess;
  const uint32_t blocks = (p.n_params + kAggThreads - 1) / kAggThreads;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(kAggThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.groups > 1) {
    cfg.gridDim = dim3(blocks, p.groups - 1, 1);
    cudaError_t e = cudaLaunchKernelEx(&cfg, group_totals_kernel, p);
    if (e != cudaSuccess) return e;
  }
  cfg.gridDim = dim3(blocks, p.groups, 1);
  return cudaLaunchKernelEx(&cfg, apply_updates_kernel, p);
}

cudaError_t launch_to_bf16(const float* src, void* dst, size_t n, cudaStream_t s) {
  if (!n) return cudaSuccess;
  size_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  to_bf16_kernel<<<(unsigned)blocks, 256, 0, s>>>(src, reinterpret_cast<__nv_bfloat16*>(dst), n);
  return cudaGetLastError();
}

}  // namespace aet
