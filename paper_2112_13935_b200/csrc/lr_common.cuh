// Pieces shared by the softmax-regression round kernels: constants of the 784 -> 10 model,
// packed-pair arithmetic, mbarrier and bulk-copy wrappers (every wait bounded), the
// transposing shuffle reductions and the hardware named barriers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace aet {
namespace lr {

constexpr int kD = 784, kC = 10, kWarps = 4, kThreads = kWarps * 32, kPix = 8;
constexpr int kLanes = 25;            // pixel groups per warp: 25+25+25+23 = 98
constexpr int kGroups = kD / kPix;    // 98
constexpr int kStages = 8;            // rows in flight
constexpr uint32_t kRowBytes = kD * sizeof(float);
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kWaitLimit = 1u << 22;  // mbarrier polls before giving up

// the blocked kernels (lambda = 0) take kM consecutive steps of the recursion at once
constexpr int kM = 8;                  // samples per block
constexpr int kCh = kC / 2;            // classes per thread
constexpr int kPairs = kM * (kM - 1) / 2;
constexpr int kParams = kD * kC + kC;                 // 7,850
constexpr int kStageFloats = (kParams + 31) / 32 * 32;   // a model row as the arrays store it (128-byte multiple)

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {  // a * b + c on both halves
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
  u64 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
  u64 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float rcp(float v) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float ex2(float v) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float shx(float v, int m) { return __shfl_xor_sync(0xffffffffu, v, m); }

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t parity, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) { return mbar_wait_limit(bar, parity, kWaitLimit); }
// One row global -> shared, 16-byte aligned on both sides, size a multiple of 16.
__device__ __forceinline__ void bulk_load_row(float* dst, const float* src, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst)), "l"(src), "r"(kRowBytes), "r"(smem_addr(bar)) : "memory");
}

// n bytes global -> shared and shared -> global (both 16-byte aligned, n a multiple of 16).
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store_and_wait(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_addr(src)), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the source may be reused after this
}

// Sum each of the 10 per-lane partials over the warp.  On return lane L holds
// the total of class lr_class(L) if lr_class_valid(L); 12 shuffles instead of 50.
__device__ __forceinline__ float reduce10(const float (&a)[kC], int lane) {
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
  float r[5];
#pragma unroll
  for (int i = 0; i < 5; ++i) {
    float keep = b4 ? a[5 + i] : a[i], send = b4 ? a[i] : a[5 + i];
    r[i] = keep + shx(send, 16);
  }
  float q0 = (b3 ? r[3] : r[0]) + shx(b3 ? r[0] : r[3], 8);
  float q1 = (b3 ? r[4] : r[1]) + shx(b3 ? r[1] : r[4], 8);
  float q2 = (b3 ? 0.f : r[2]) + shx(b3 ? r[2] : 0.f, 8);
  float p0 = (b2 ? q2 : q0) + shx(b2 ? q0 : q2, 4);
  float p1 = (b2 ? 0.f : q1) + shx(b2 ? q1 : 0.f, 4);
  float o = (b1 ? p1 : p0) + shx(b1 ? p0 : p1, 2);
  return o + shx(o, 1);
}
__device__ __forceinline__ int lr_class(int lane) {
  return ((lane & 16) ? 5 : 0) + ((lane & 8) ? 3 : 0) + ((lane & 4) ? 2 : 0) + ((lane & 2) ? 1 : 0);
}
__device__ __forceinline__ bool lr_class_valid(int lane) {
  const bool b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
  return (b3 ? !b2 : !(b2 && b1)) && !(lane & 1);
}

// One stage of a transposing reduction: N values per lane in, ceil(N/2) out; the
// lane keeps the half selected by its `bit` and receives the partner's other half.
template <int N>
__device__ __forceinline__ void bfly_stage(const float (&v)[N], float (&o)[(N + 1) / 2], int mask, bool bit) {
  constexpr int H = (N + 1) / 2;
#pragma unroll
  for (int i = 0; i < H; ++i) {
    const float lo = v[i];
    const float hi = (i + H < N) ? v[(i + H < N) ? i + H : 0] : 0.f;
    const float keep = bit ? hi : lo, send = bit ? lo : hi;
    o[i] = keep + __shfl_xor_sync(0xffffffffu, send, mask);
  }
}
template <int N> struct BflyDims {
  static constexpr int n1 = (N + 1) / 2, n2 = (n1 + 1) / 2, n3 = (n2 + 1) / 2, n4 = (n3 + 1) / 2, n5 = (n4 + 1) / 2;
};
// Sums v[i] over the 32 lanes for every i; lane L ends with n5 totals in o[].
template <int N>
__device__ __forceinline__ void bfly_reduce5(const float (&v)[N], float (&o)[BflyDims<N>::n5], int lane) {
  typedef BflyDims<N> D;
  float a[D::n1], b[D::n2], c[D::n3], d[D::n4];
  bfly_stage<N>(v, a, 16, lane & 16);
  bfly_stage<D::n1>(a, b, 8, lane & 8);
  bfly_stage<D::n2>(b, c, 4, lane & 4);
  bfly_stage<D::n3>(c, d, 2, lane & 2);
  bfly_stage<D::n4>(d, o, 1, lane & 1);
}
// Which v[] index the lane's i-th total belongs to (-1: padding).
template <int N>
__device__ __forceinline__ int bfly_index5(int lane, int i) {
  typedef BflyDims<N> D;
  const int i4 = i + ((lane & 1) ? D::n5 : 0);
  const int i3 = i4 + ((lane & 2) ? D::n4 : 0);
  const int i2 = i3 + ((lane & 4) ? D::n3 : 0);
  const int i1 = i2 + ((lane & 8) ? D::n2 : 0);
  const int i0 = i1 + ((lane & 16) ? D::n1 : 0);
  const bool ok = i4 < D::n4 && i3 < D::n3 && i2 < D::n2 && i1 < D::n1 && i0 < N;
  return ok ? i0 : -1;
}
// The same over the 16 lanes that share bit 0 (masks 16, 8, 4, 2): n4 totals per lane.
template <int N>
__device__ __forceinline__ void bfly_reduce4(const float (&v)[N], float (&o)[BflyDims<N>::n4], int lane) {
  typedef BflyDims<N> D;
  float a[D::n1], b[D::n2], c[D::n3];
  bfly_stage<N>(v, a, 16, lane & 16);
  bfly_stage<D::n1>(a, b, 8, lane & 8);
  bfly_stage<D::n2>(b, c, 4, lane & 4);
  bfly_stage<D::n3>(c, o, 2, lane & 2);
}
template <int N>
__device__ __forceinline__ int bfly_index4(int lane, int i) {
  typedef BflyDims<N> D;
  const int i3 = i + ((lane & 2) ? D::n4 : 0);
  const int i2 = i3 + ((lane & 4) ? D::n3 : 0);
  const int i1 = i2 + ((lane & 8) ? D::n2 : 0);
  const int i0 = i1 + ((lane & 16) ? D::n1 : 0);
  const bool ok = i3 < D::n3 && i2 < D::n2 && i1 < D::n1 && i0 < N;
  return ok ? i0 : -1;
}
__device__ __forceinline__ constexpr int pair_index(int s, int t) { return t * (t - 1) / 2 + s; }  // s < t

__device__ __forceinline__ void named_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }


}  // namespace lr
}  // namespace aet
