// Local-SGD round of one client for softmax regression 784 -> 10, batch 1.
//
// Algorithm 3, MainComputeNode, inner loop: "sample xi; g = grad f(w_c, xi);
// w_c -= eta_i * g; U_i += g; h++" repeated s_{i,c} times, then the tuple
// (c, U_i, i) is sent.  One CTA runs one round-task; the client's model and
// the running update sum stay in registers for the whole round and only the
// sampled rows stream in from HBM.
//
// Work split: 7 warps x 28 lanes = 196 threads, thread u owns pixels 4u..4u+3
// and all 10 classes of them (40 weights + 40 update-sum entries).  Per sample:
//   1. every thread loads its 16 bytes of the row (prefetched kDepth samples
//      ahead, straight into registers; the index stream is a counter hash, so
//      addresses are known in advance);
//   2. 40 FMAs give the thread's share of the 10 logits;
//   3. a transposing butterfly (12 shuffles) leaves each class total of the warp
//      in one lane; those go to shared memory, one barrier;
//   4. every warp redundantly sums the 7 partials, does the softmax across its
//      lanes and broadcasts delta = p - onehot(y);
//   5. 80 FMAs update W and U.
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"

namespace aet {
namespace {

constexpr int kD = 784, kC = 10, kWarps = 7, kLanes = 28, kThreads = kWarps * 32, kPix = 4;
constexpr int kDepth = 4;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float4 ld_row(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ float shx(float v, int m) { return __shfl_xor_sync(0xffffffffu, v, m); }

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

template <bool kL2>
__global__ void __launch_bounds__(kThreads) lr_round_kernel(RoundLaunch p) {
  __shared__ float part[2][kWarps][16];

  const TaskDesc t = p.tasks[p.task_begin + blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool active = lane < kLanes;
  const int u = warp * kLanes + (active ? lane : 0);  // pixel group
  const int cls = lane & 15;                            // class this lane handles in the softmax
  const bool cls_ok = cls < kC;

  // ---- start model: server snapshot minus own update sums still in flight ----
  float W[kPix][kC], U[kPix][kC];
  float bias = 0.f, ubias = 0.f;
  {
    const float* src = p.snaps + (size_t)t.snap_slot * p.stride;
    const float4* s4 = reinterpret_cast<const float4*>(src + (size_t)u * (kPix * kC));
    float* w = &W[0][0];
#pragma unroll
    for (int j = 0; j < kPix * kC / 4; ++j) {
      float4 v = active ? __ldg(s4 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
      w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
    }
    if (cls_ok) bias = __ldg(src + kD * kC + cls);
    for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
      const InflightRef ref = p.inflight[t.inflight_off + f];
      const float* us = p.U + (size_t)ref.seq * p.stride;
      const float4* u4 = reinterpret_cast<const float4*>(us + (size_t)u * (kPix * kC));
#pragma unroll
      for (int j = 0; j < kPix * kC / 4; ++j) {
        float4 v = active ? __ldg(u4 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        w[4 * j] = fmaf(-ref.eta, v.x, w[4 * j]);
        w[4 * j + 1] = fmaf(-ref.eta, v.y, w[4 * j + 1]);
        w[4 * j + 2] = fmaf(-ref.eta, v.z, w[4 * j + 2]);
        w[4 * j + 3] = fmaf(-ref.eta, v.w, w[4 * j + 3]);
      }
      if (cls_ok) bias = fmaf(-ref.eta, __ldg(us + kD * kC + cls), bias);
    }
#pragma unroll
    for (int a = 0; a < kPix; ++a)
#pragma unroll
      for (int k = 0; k < kC; ++k) U[a][k] = 0.f;
  }

  const ClientData cd = p.clients[t.client];
  const uint64_t key = p.sample_keys[t.client];
  const float4* rows = reinterpret_cast<const float4*>(cd.x);
  const float eta = t.eta;
  const float decay = p.l2;  // lambda

  // ---- prefetch ring ----
  float4 xq[kDepth];
  int yq[kDepth];
  const uint32_t n = t.n_samples;
  uint32_t h = 0;  // local iteration counter of Algorithm 3
#pragma unroll
  for (int dpt = 0; dpt < kDepth; ++dpt) {
    xq[dpt] = make_float4(0.f, 0.f, 0.f, 0.f);
    yq[dpt] = 0;
    if ((uint32_t)dpt < n) {
      const uint32_t idx = sample_index(draw(key, t.sample_ctr0 + dpt), cd.n);
      if (active) xq[dpt] = ld_row(rows + (size_t)idx * (kD / 4) + u);
      yq[dpt] = __ldg(cd.y + idx);
    }
  }

  for (uint32_t base = 0; base < n; base += kDepth) {
#pragma unroll
    for (int dpt = 0; dpt < kDepth; ++dpt) {
      const uint32_t k = base + dpt;
      if (k >= n) break;
      const float4 xv = xq[dpt];
      const int y = yq[dpt];
      // refill this slot with sample k + kDepth
      if (k + kDepth < n) {
        const uint32_t idx = sample_index(draw(key, t.sample_ctr0 + k + kDepth), cd.n);
        if (active) xq[dpt] = ld_row(rows + (size_t)idx * (kD / 4) + u);
        yq[dpt] = __ldg(cd.y + idx);
      }
      const float x[kPix] = {xv.x, xv.y, xv.z, xv.w};

      float acc[kC];
#pragma unroll
      for (int c = 0; c < kC; ++c) acc[c] = x[0] * W[0][c];
#pragma unroll
      for (int a = 1; a < kPix; ++a)
#pragma unroll
        for (int c = 0; c < kC; ++c) acc[c] = fmaf(x[a], W[a][c], acc[c]);

      const float tot = reduce10(acc, lane);
      const int buf = k & 1;
      if (lr_class_valid(lane)) part[buf][warp][lr_class(lane)] = tot;
      __syncthreads();

      float z = bias;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) z += part[buf][w][cls];
      z = cls_ok ? z : -INFINITY;
      float m = z;
      m = fmaxf(m, shx(m, 8)); m = fmaxf(m, shx(m, 4));
      m = fmaxf(m, shx(m, 2)); m = fmaxf(m, shx(m, 1));
      const float e = exp2f((z - m) * kLog2e);
      float sum = e;
      sum += shx(sum, 8); sum += shx(sum, 4); sum += shx(sum, 2); sum += shx(sum, 1);
      const float delta = cls_ok ? __fdividef(e, sum) - (cls == y ? 1.f : 0.f) : 0.f;
      bias = fmaf(-eta, delta, bias);
      ubias += delta;
      ++h;

      float d[kC];
#pragma unroll
      for (int c = 0; c < kC; ++c) d[c] = __shfl_sync(0xffffffffu, delta, c);
#pragma unroll
      for (int a = 0; a < kPix; ++a)
#pragma unroll
        for (int c = 0; c < kC; ++c) {
          if (kL2) {
            const float g = fmaf(d[c], x[a], decay * W[a][c]);
            W[a][c] = fmaf(-eta, g, W[a][c]);
            U[a][c] += g;
          } else {
            W[a][c] = fmaf(-eta * d[c], x[a], W[a][c]);
            U[a][c] = fmaf(d[c], x[a], U[a][c]);
          }
        }
    }
  }

  // ---- event trigger: h reached s_{i,c}; publish U_i (and the end model) ----
  {
    float* dstU = p.U + (size_t)t.seq * p.stride;
    if (active) {
      float4* d4 = reinterpret_cast<float4*>(dstU + (size_t)u * (kPix * kC));
      const float* us = &U[0][0];
#pragma unroll
      for (int j = 0; j < kPix * kC / 4; ++j)
        d4[j] = make_float4(us[4 * j], us[4 * j + 1], us[4 * j + 2], us[4 * j + 3]);
    }
    if (warp == 0 && lane < kC) dstU[kD * kC + lane] = ubias;
    if (p.w_end) {
      float* dstW = p.w_end + (size_t)t.seq * p.stride;
      if (active) {
        float4* d4 = reinterpret_cast<float4*>(dstW + (size_t)u * (kPix * kC));
        const float* ws = &W[0][0];
#pragma unroll
        for (int j = 0; j < kPix * kC / 4; ++j)
          d4[j] = make_float4(ws[4 * j], ws[4 * j + 1], ws[4 * j + 2], ws[4 * j + 3]);
      }
      if (warp == 0 && lane < kC) dstW[kD * kC + lane] = bias;
    }
    if (threadIdx.x == 0) {
      TriggerRec rec;
      rec.client = t.client; rec.round = t.round; rec.samples_done = h; rec.flags = 1;
      p.trig[t.seq] = rec;
    }
  }
}

}  // namespace

cudaError_t launch_lr_rounds(const RoundLaunch& p, cudaStream_t s) {
  if (p.n_tasks == 0) return cudaSuccess;
  if (p.l2 != 0.f)
    lr_round_kernel<true><<<p.n_tasks, kThreads, 0, s>>>(p);
  else
    lr_round_kernel<false><<<p.n_tasks, kThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace aet
