// Local-SGD round of one client for softmax regression 784 -> 10, batch 1.
//
// Algorithm 3, MainComputeNode, inner loop: "sample xi; g = grad f(w_c, xi);
// w_c -= eta_i * g; U_i += g; h++" repeated s_{i,c} times, then the tuple
// (c, U_i, i) is sent.  One CTA runs one round-task; the client's model and
// the running update sum stay in registers for the whole round and only the
// sampled rows stream in from HBM.
//
// Work split: 4 warps (one per SM sub-partition), 98 threads own 8 consecutive
// pixels each and all 10 classes of them: 80 weights + 80 update-sum entries,
// held as 2 x 40 packed fp32 pairs (class 2c, 2c+1) so that logits and updates
// run on fma.rn.f32x2.  Per sample:
//   1. the row (3,136 B) was fetched kStages samples ahead by a bulk async copy
//      (cp.async.bulk) into a shared-memory ring, completion on an mbarrier; the
//      index stream is a counter hash, so addresses are known in advance;
//   2. 40 packed FMAs give the thread's share of the 10 logits;
//   3. a transposing butterfly (12 shuffles) leaves each class total of the warp
//      in one lane; 4 x 10 partials go to shared memory, one barrier;
//   4. every thread sums the partials and computes the softmax itself on packed
//      pairs (no further shuffles on the critical path): delta = p - onehot(y);
//      the bias is one more always-1 "pixel" owned by a spare lane;
//   5. 80 packed FMAs update W and U.
// Two CTAs fit on one SM (<= 255 registers), so with many clients one CTA's
// latency-bound phases overlap the other's FMA phases.
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"

namespace aet {
namespace {

constexpr int kD = 784, kC = 10, kWarps = 4, kThreads = kWarps * 32, kPix = 8;
constexpr int kLanes = 25;            // pixel groups per warp: 25+25+25+23 = 98
constexpr int kGroups = kD / kPix;    // 98
constexpr int kStages = 8;            // rows in flight
constexpr uint32_t kRowBytes = kD * sizeof(float);
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kWaitLimit = 1u << 22;  // mbarrier polls before giving up

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

// kShared: one warp (rotating) computes the softmax and hands delta to the others
// through shared memory (a second barrier): fewer instructions per sample, more
// latency - used when enough CTAs share an SM to hide it.
template <bool kL2, bool kShared>
__global__ void __launch_bounds__(kThreads, 2) lr_round_kernel(RoundLaunch p) {
  __shared__ __align__(128) float rows[kStages][kD];
  __shared__ __align__(16) float part[2][kWarps][12];  // class totals per warp, double-buffered
  __shared__ __align__(16) float onehot[kC][12];        // row y: -1 at class y, else 0
  __shared__ __align__(16) float dsm[2][12];            // delta of the current sample (kShared)
  __shared__ __align__(8) uint64_t full[kStages];

  const TaskDesc t = p.tasks[p.task_begin + blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int u_raw = warp * kLanes + lane;
  const bool active = lane < kLanes && u_raw < kGroups;
  // The bias rides along as one more "pixel" that is always 1: the first spare
  // lane of the last warp holds it in row 0 of its (otherwise zero) weights, so
  // logits, update and update sum need no code of their own.
  const bool is_bias = warp == kWarps - 1 && u_raw == kGroups;
  const int u = active ? u_raw : 0;

  const ClientData cd = p.clients[t.client];
  const uint64_t key = p.sample_keys[t.client];
  const float* xrows = reinterpret_cast<const float*>(cd.x);
  const uint32_t n = t.n_samples;
  const float eta = t.eta;

  if (threadIdx.x == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kC * 12) onehot[threadIdx.x / 12][threadIdx.x % 12] = (threadIdx.x / 12 == threadIdx.x % 12) ? -1.f : 0.f;
  if (threadIdx.x < 2 * kWarps * 12) (&part[0][0][0])[threadIdx.x] = 0.f;
  if (threadIdx.x < 24) (&dsm[0][0])[threadIdx.x] = 0.f;

  // Sample indices and labels, 32 samples per block, lane l holds sample blk*32+l.
  auto block_idx = [&](uint32_t first) -> uint32_t {
    const uint32_t k = first + lane;
    return k < n ? sample_index(draw(key, t.sample_ctr0 + k), cd.n) : 0u;
  };
  uint32_t idx_cur = block_idx(0), idx_nxt = block_idx(32);
  int y_cur = __ldg(cd.y + idx_cur), y_nxt = __ldg(cd.y + idx_nxt);
  __syncthreads();

  // prologue: fill the ring
  if (warp == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) {
      const uint32_t idx = __shfl_sync(0xffffffffu, idx_cur, s);
      if (lane == 0 && (uint32_t)s < n) {
        mbar_expect_tx(&full[s], kRowBytes);
        bulk_load_row(rows[s], xrows + (size_t)idx * kD, &full[s]);
      }
    }
  }

  // ---- start model: server snapshot minus own update sums still in flight ----
  u64 W2[kPix][kC / 2], U2[kPix][kC / 2];
  {
    const float* src = p.snaps + (size_t)t.snap_slot * p.stride;
    // a pixel group reads 80 consecutive floats; the bias lane reads the 10 biases into row 0
    const float2* s2 = reinterpret_cast<const float2*>(src + (is_bias ? (size_t)kD * kC : (size_t)u * (kPix * kC)));
#pragma unroll
    for (int a = 0; a < kPix; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) {
        const bool live = active || (is_bias && a == 0);
        float2 v = live ? __ldg(s2 + a * (kC / 2) + c) : make_float2(0.f, 0.f);
        W2[a][c] = pack2(v.x, v.y);
        U2[a][c] = 0ull;
      }
    for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
      const InflightRef ref = p.inflight[t.inflight_off + f];
      const float* us = p.U + (size_t)ref.seq * p.stride;
      const float2* u2 = reinterpret_cast<const float2*>(us + (is_bias ? (size_t)kD * kC : (size_t)u * (kPix * kC)));
      const u64 ne = pack2(-ref.eta, -ref.eta);
#pragma unroll
      for (int a = 0; a < kPix; ++a)
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) {
          const bool live = active || (is_bias && a == 0);
          float2 v = live ? __ldg(u2 + a * (kC / 2) + c) : make_float2(0.f, 0.f);
          W2[a][c] = fma2(ne, pack2(v.x, v.y), W2[a][c]);
        }
    }
  }

  const u64 neta2 = pack2(-eta, -eta);
  const u64 log2e2 = pack2(kLog2e, kLog2e);
  const float lam = is_bias ? 0.f : p.l2;   // no l2 term on the bias
  const u64 lam2 = pack2(lam, lam);
  const u64 nel2 = pack2(-eta * lam, -eta * lam);
  uint32_t h = 0;  // local iteration counter of Algorithm 3
  bool timed_out = false;
  uint32_t timeout_at = 0;

  for (uint32_t k = 0; k < n; ++k) {
    const int slot = k & (kStages - 1);
    const int buf = k & 1;
    if ((k & 31) == 0 && k) {  // next block of indices / labels
      idx_cur = idx_nxt;
      y_cur = y_nxt;
      idx_nxt = block_idx(k + 32);
      y_nxt = __ldg(cd.y + idx_nxt);
    }
    const int y = __shfl_sync(0xffffffffu, y_cur, k & 31);
    // index of the row that will take this slot once everybody has read it
    const uint32_t kn = k + kStages;
    uint32_t idx_next = 0;
    if (warp == 0) idx_next = __shfl_sync(0xffffffffu, (kn >> 5) == (k >> 5) ? idx_cur : idx_nxt, kn & 31);

    const bool landed = mbar_wait(&full[slot], (k / kStages) & 1);

    float4 xa = make_float4(is_bias ? 1.f : 0.f, 0.f, 0.f, 0.f), xb = make_float4(0.f, 0.f, 0.f, 0.f);
    if (active) {
      const float4* r4 = reinterpret_cast<const float4*>(&rows[slot][u * kPix]);
      xa = r4[0];
      xb = r4[1];
    }
    const float x[kPix] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
    u64 xx[kPix];
#pragma unroll
    for (int a = 0; a < kPix; ++a) xx[a] = pack2(x[a], x[a]);

    // logits: this thread's share
    u64 acc2[kC / 2];
#pragma unroll
    for (int c = 0; c < kC / 2; ++c) acc2[c] = mul2(xx[0], W2[0][c]);
#pragma unroll
    for (int a = 1; a < kPix; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) acc2[c] = fma2(xx[a], W2[a][c], acc2[c]);
    float acc[kC];
#pragma unroll
    for (int c = 0; c < kC / 2; ++c) unpack2(acc2[c], acc[2 * c], acc[2 * c + 1]);

    const float tot = reduce10(acc, lane);
    if (lr_class_valid(lane)) part[buf][warp][lr_class(lane)] = tot;
    // partials visible; every thread has read its pixels of this row.  The same
    // barrier carries the verdict of the bounded wait so that all threads leave together.
    if (__syncthreads_or(!landed)) { timed_out = true; timeout_at = k; break; }

    if (threadIdx.x == 0 && kn < n) {
      mbar_expect_tx(&full[slot], kRowBytes);
      bulk_load_row(rows[slot], xrows + (size_t)idx_next * kD, &full[slot]);
    }

    u64 d2[kC / 2], nd2[kC / 2];
    if (kShared) {
      if (warp == (int)(k & (kWarps - 1))) {
        const int cls = lane & 15;
        float z = -INFINITY;
        if (cls < kC) z = (part[buf][0][cls] + part[buf][1][cls]) + (part[buf][2][cls] + part[buf][3][cls]);
        float m = z;
        m = fmaxf(m, shx(m, 8)); m = fmaxf(m, shx(m, 4)); m = fmaxf(m, shx(m, 2)); m = fmaxf(m, shx(m, 1));
        const float e = ex2((z - m) * kLog2e);
        float sum = e;
        sum += shx(sum, 8); sum += shx(sum, 4); sum += shx(sum, 2); sum += shx(sum, 1);
        if (lane < kC) dsm[buf][lane] = fmaf(e, rcp(sum), lane == y ? -1.f : 0.f);
      }
      __syncthreads();
      const ulonglong2* dq = reinterpret_cast<const ulonglong2*>(&dsm[buf][0]);
      const ulonglong2 q0 = dq[0], q1 = dq[1], q2 = dq[2];
      d2[0] = q0.x; d2[1] = q0.y; d2[2] = q1.x; d2[3] = q1.y; d2[4] = q2.x;
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) nd2[c] = mul2(d2[c], neta2);
    } else {
    // softmax over the 10 logits, computed by every thread on packed pairs
    u64 z2[6];
    {
      const ulonglong2* q = reinterpret_cast<const ulonglong2*>(&part[buf][0][0]);
      u64 s01[6], s23[6];
#pragma unroll
      for (int j = 0; j < 3; ++j) {
        const ulonglong2 a0 = q[j], a1 = q[3 + j], a2 = q[6 + j], a3 = q[9 + j];
        s01[2 * j] = add2(a0.x, a1.x); s01[2 * j + 1] = add2(a0.y, a1.y);
        s23[2 * j] = add2(a2.x, a3.x); s23[2 * j + 1] = add2(a2.y, a3.y);
      }
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) z2[c] = add2(s01[c], s23[c]);
    }
    float z[kC];
#pragma unroll
    for (int c = 0; c < kC / 2; ++c) unpack2(z2[c], z[2 * c], z[2 * c + 1]);
    const float m = fmaxf(fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7]))),
                          fmaxf(z[8], z[9]));
    const float nms = -m * kLog2e;
    const u64 nms2 = pack2(nms, nms);
    u64 e2[kC / 2];
#pragma unroll
    for (int c = 0; c < kC / 2; ++c) {
      float lo, hi;
      unpack2(fma2(z2[c], log2e2, nms2), lo, hi);
      e2[c] = pack2(ex2(lo), ex2(hi));
    }
    float slo, shi;
    unpack2(add2(add2(add2(e2[0], e2[1]), add2(e2[2], e2[3])), e2[4]), slo, shi);
    const float inv = rcp(slo + shi);
    const u64 inv2 = pack2(inv, inv);
    {
      const ulonglong2* oh = reinterpret_cast<const ulonglong2*>(&onehot[y][0]);
      const ulonglong2 o0 = oh[0], o1 = oh[1], o2 = oh[2];
      d2[0] = fma2(e2[0], inv2, o0.x); d2[1] = fma2(e2[1], inv2, o0.y);
      d2[2] = fma2(e2[2], inv2, o1.x); d2[3] = fma2(e2[3], inv2, o1.y);
      d2[4] = fma2(e2[4], inv2, o2.x);
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) nd2[c] = mul2(d2[c], neta2);
    }
    }
    ++h;

    // W -= eta * g, U += g with g = delta x^T (+ lambda W)
#pragma unroll
    for (int a = 0; a < kPix; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) {
        if (kL2) {
          const u64 w_old = W2[a][c];
          U2[a][c] = fma2(xx[a], d2[c], U2[a][c]);
          U2[a][c] = fma2(w_old, lam2, U2[a][c]);
          W2[a][c] = fma2(xx[a], nd2[c], w_old);
          W2[a][c] = fma2(w_old, nel2, W2[a][c]);
        } else {
          W2[a][c] = fma2(xx[a], nd2[c], W2[a][c]);
          U2[a][c] = fma2(xx[a], d2[c], U2[a][c]);
        }
      }
  }

  if (timed_out) {
    // A row never arrived.  Flag it, give copies still in flight a bounded
    // chance to land (their target is this CTA's shared memory), and leave.
    if (threadIdx.x == 0) {
      if (p.status) atomicOr(p.status, 1u);
      for (uint32_t j = timeout_at; j < n && j < timeout_at + kStages; ++j)
        mbar_wait(&full[j & (kStages - 1)], (j / kStages) & 1);
    }
    return;
  }

  // ---- event trigger: h reached s_{i,c}; publish U_i (and the end model) ----
  {
    const size_t off = is_bias ? (size_t)kD * kC : (size_t)u * (kPix * kC);
    float2* dU = reinterpret_cast<float2*>(p.U + (size_t)t.seq * p.stride + off);
    float2* dW = p.w_end ? reinterpret_cast<float2*>(p.w_end + (size_t)t.seq * p.stride + off) : nullptr;
#pragma unroll
    for (int a = 0; a < kPix; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) {
        if (active || (is_bias && a == 0)) {
          float lo, hi;
          unpack2(U2[a][c], lo, hi);
          dU[a * (kC / 2) + c] = make_float2(lo, hi);
          if (dW) {
            unpack2(W2[a][c], lo, hi);
            dW[a * (kC / 2) + c] = make_float2(lo, hi);
          }
        }
      }
    if (threadIdx.x == 0) {
      TriggerRec rec;
      rec.client = t.client; rec.round = t.round; rec.samples_done = h; rec.flags = 1;
      p.trig[t.seq] = rec;
    }
  }
}

// ---------------------------------------------------------------------------
// Blocked form of the same recursion for lambda = 0.
//
// kM consecutive batch-1 steps of Algorithm 3 ("g = grad f(w_c, xi); w_c -=
// eta_i g; U_i += g") are taken together.  With W the model at the start of the
// block, delta_s = softmax(z_s) - onehot(y_s) and G[s][t] = x_s . x_t + 1 (the
// 1 is the bias), step t of the block sees the logits
//     z_t = W x_t + b - eta * sum_{s<t} delta_s G[s][t],
// because W_t = W - eta * sum_{s<t} delta_s x_s^T.  So per block:
//   P1  Z0 = W X (every thread: its 7 pixels x 10 classes x kM samples), summed
//       over the CTA by a transposing shuffle butterfly and 4 partials in shared
//       memory;
//   R   one warp (rotating) walks the kM samples: lane t owns sample t, takes the
//       softmax of its corrected logits and hands -eta*delta_t to the later
//       samples' lanes by shuffle; delta and -eta*delta go to shared memory;
//       meanwhile the other three warps compute the Gram matrix of the NEXT block
//       (it does not depend on W) and one of them issues the bulk copies of the
//       block after that;
//   P3  W += (-eta delta_t) x_t^T and U += delta_t x_t^T for the block's samples.
// The result equals the step-by-step recursion up to fp32 rounding order.  One
// barrier pair per kM samples instead of one per sample, and the latency-bound
// softmax chain of one block overlaps the FMA phases of the CTA sharing the SM.
//
// Work split: 4 warps x 28 lanes x 7 consecutive pixels = 784; lane 28 of the
// last warp carries the bias as an always-1 pixel.  W and U stay in registers
// (2 x 35 packed pairs).  Rows arrive by cp.async.bulk into a ring of 3 blocks,
// issued two blocks ahead; every mbarrier wait is bounded.
constexpr int kM = 8;                  // samples per block
constexpr int kSlots = 3;              // blocks of rows in shared memory
constexpr int kPx = 7, kAct = 28;      // pixels per thread, pixel-owning lanes per warp
constexpr int kQ = 4;                  // samples per accumulator group in P1
constexpr int kPairs = kM * (kM - 1) / 2;
static_assert(kAct * kWarps * kPx == kD, "pixel split");
static_assert(kM % kQ == 0 && kM <= 8, "block shape");

struct __align__(128) BlkSmem {
  float rows[kSlots][kM][kD];
  float partZ[kWarps][kM * kC];       // per-warp totals of Z0, index t*10 + c
  float partG[2][kWarps][32];         // per-warp totals of the Gram pairs, double-buffered by block parity
  float dbuf[kM][24];                 // [0..9] delta_t, [12..21] -eta*delta_t
  float onehot[kC][12];               // row y: -1 at class y, else 0
  float consts[16];                   // [0..6] = 1,0,0,0,0,0,0 (bias lane's "row"); [8..14] = 0 (idle lanes)
  int ys[kSlots][kM];
  uint64_t full[kSlots];
};

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
__device__ __forceinline__ void bfly_reduce(const float (&v)[N], float (&o)[BflyDims<N>::n5], int lane) {
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
__device__ __forceinline__ int bfly_index(int lane, int i) {
  typedef BflyDims<N> D;
  const int i4 = i + ((lane & 1) ? D::n5 : 0);
  const int i3 = i4 + ((lane & 2) ? D::n4 : 0);
  const int i2 = i3 + ((lane & 4) ? D::n3 : 0);
  const int i1 = i2 + ((lane & 8) ? D::n2 : 0);
  const int i0 = i1 + ((lane & 16) ? D::n1 : 0);
  const bool ok = i4 < D::n4 && i3 < D::n3 && i2 < D::n2 && i1 < D::n1 && i0 < N;
  return ok ? i0 : -1;
}
__device__ __forceinline__ constexpr int pair_index(int s, int t) { return t * (t - 1) / 2 + s; }  // s < t

__global__ void __launch_bounds__(kThreads, 2) lr_block_kernel(RoundLaunch p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  BlkSmem& sm = *reinterpret_cast<BlkSmem*>(smem_raw);

  const TaskDesc t = p.tasks[p.task_begin + blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool active = lane < kAct;
  const bool is_bias = warp == kWarps - 1 && lane == kAct;
  const int g = warp * kAct + (active ? lane : 0);   // pixel group: pixels 7g .. 7g+6

  const ClientData cd = p.clients[t.client];
  const uint64_t key = p.sample_keys[t.client];
  const float* xrows = reinterpret_cast<const float*>(cd.x);
  const uint32_t n = t.n_samples;
  const uint32_t nblk = (n + kM - 1) / kM;
  const float eta = t.eta;

  if (threadIdx.x == 0) {
#pragma unroll
    for (int s = 0; s < kSlots; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kC * 12) sm.onehot[threadIdx.x / 12][threadIdx.x % 12] = (threadIdx.x / 12 == threadIdx.x % 12) ? -1.f : 0.f;
  if (threadIdx.x < 16) sm.consts[threadIdx.x] = threadIdx.x == 0 ? 1.f : 0.f;
  __syncthreads();

  // Producer step: the rows and labels of block kb into ring slot kb % kSlots.
  auto produce = [&](uint32_t kb) {
    const int sb = kb % kSlots;
    const uint32_t nvb = min((uint32_t)kM, n - kb * kM);
    if (lane == 0) mbar_expect_tx(&sm.full[sb], nvb * kRowBytes);
    __syncwarp();
    if ((uint32_t)lane < nvb) {
      const uint32_t idx = sample_index(draw(key, t.sample_ctr0 + kb * kM + lane), cd.n);
      bulk_load_row(sm.rows[sb][lane], xrows + (size_t)idx * kD, &sm.full[sb]);
      sm.ys[sb][lane] = __ldg(cd.y + idx);
    }
  };
  if (warp == 0) {
    produce(0);
    if (nblk > 1) produce(1);
  }

  // ---- start model: server snapshot minus own update sums still in flight ----
  u64 W2[kPx][kC / 2], U2[kPx][kC / 2];
  const bool owns = active || is_bias;
  const size_t poff = is_bias ? (size_t)kD * kC : (size_t)g * (kPx * kC);
  {
    const float2* s2 = reinterpret_cast<const float2*>(p.snaps + (size_t)t.snap_slot * p.stride + poff);
#pragma unroll
    for (int a = 0; a < kPx; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) {
        const bool live = active || (is_bias && a == 0);
        const float2 v = live ? __ldg(s2 + a * (kC / 2) + c) : make_float2(0.f, 0.f);
        W2[a][c] = pack2(v.x, v.y);
        U2[a][c] = 0ull;
      }
    for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
      const InflightRef ref = p.inflight[t.inflight_off + f];
      const float2* u2 = reinterpret_cast<const float2*>(p.U + (size_t)ref.seq * p.stride + poff);
      const u64 ne = pack2(-ref.eta, -ref.eta);
#pragma unroll
      for (int a = 0; a < kPx; ++a)
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) {
          const bool live = active || (is_bias && a == 0);
          const float2 v = live ? __ldg(u2 + a * (kC / 2) + c) : make_float2(0.f, 0.f);
          W2[a][c] = fma2(ne, pack2(v.x, v.y), W2[a][c]);
        }
    }
  }

  // Where this thread reads "its pixels" of sample (slot, t): pixel-owning lanes
  // from the row, the bias lane from {1,0,...}, idle lanes from zeros (row stride 0).
  const float* xbase = active ? &sm.rows[0][0][g * kPx] : (is_bias ? &sm.consts[0] : &sm.consts[8]);
  const int rs = active ? kD : 0;

  // where the lane's butterfly totals go
  int zidx[2], gidx;
  zidx[0] = bfly_index<kQ * kC>(lane, 0);
  zidx[1] = bfly_index<kQ * kC>(lane, 1);
  gidx = bfly_index<kPairs>(lane, 0);
  static_assert(BflyDims<kQ * kC>::n5 == 2 && BflyDims<kPairs>::n5 == 1, "butterfly widths");

  // Gram pairs of block kb over this warp's share of the pixels (rank r of 3).
  auto gram_partial = [&](uint32_t kb, int r) {
    const float* rb = &sm.rows[kb % kSlots][0][0];
    float gacc[kPairs];
#pragma unroll
    for (int i = 0; i < kPairs; ++i) gacc[i] = 0.f;
    for (int chunk = r; chunk * 32 < kD; chunk += 3) {
      const int px = chunk * 32 + lane;
      if (px < kD) {
        float x[kM];
#pragma unroll
        for (int s = 0; s < kM; ++s) x[s] = rb[s * kD + px];
#pragma unroll
        for (int b = 1; b < kM; ++b)
#pragma unroll
          for (int a = 0; a < b; ++a) gacc[pair_index(a, b)] = fmaf(x[a], x[b], gacc[pair_index(a, b)]);
      }
    }
    float o[1];
    bfly_reduce<kPairs>(gacc, o, lane);
    if (gidx >= 0) sm.partG[kb & 1][warp][gidx] = o[0];
  };

  const u64 neta2 = pack2(-eta, -eta);
  const u64 log2e2 = pack2(kLog2e, kLog2e);
  bool ok = true;
  bool timed_out = false;
  uint32_t timeout_at = 0;

  // Gram matrix of block 0: warps 0..2 (the rotation below treats warp 3 as busy before block 0)
  if (warp != kWarps - 1) {
    ok = mbar_wait(&sm.full[0], 0);
    gram_partial(0, warp);
  }

  for (uint32_t k = 0; k < nblk; ++k) {
    const int slot = k % kSlots;
    const uint32_t nv = min((uint32_t)kM, n - k * kM);
    ok = mbar_wait(&sm.full[slot], (k / kSlots) & 1) && ok;
    const float* xslot = xbase + (size_t)slot * kM * rs;

    // ---- P1: this thread's share of Z0 = W X, kQ samples at a time ----
#pragma unroll
    for (int q = 0; q < kM / kQ; ++q) {
      u64 acc[kQ][kC / 2];
#pragma unroll
      for (int a = 0; a < kPx; ++a)
#pragma unroll
        for (int s = 0; s < kQ; ++s) {
          const float x = xslot[(q * kQ + s) * rs + a];
          const u64 xs = pack2(x, x);
#pragma unroll
          for (int c = 0; c < kC / 2; ++c) acc[s][c] = a == 0 ? mul2(xs, W2[0][c]) : fma2(xs, W2[a][c], acc[s][c]);
        }
      float v[kQ * kC];
#pragma unroll
      for (int s = 0; s < kQ; ++s)
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) unpack2(acc[s][c], v[s * kC + 2 * c], v[s * kC + 2 * c + 1]);
      float o[2];
      bfly_reduce<kQ * kC>(v, o, lane);
      if (zidx[0] >= 0) sm.partZ[warp][q * kQ * kC + zidx[0]] = o[0];
      if (zidx[1] >= 0) sm.partZ[warp][q * kQ * kC + zidx[1]] = o[1];
    }
    // barrier A: partials visible, rows of block k-1 no longer read by anyone; it
    // also carries the verdict of the bounded waits so that all threads leave together
    if (__syncthreads_or(!ok)) { timed_out = true; timeout_at = k; break; }

    const int rwarp = k & (kWarps - 1);
    if (warp == rwarp) {
      // ---- R: the block's kM dependent softmax steps, lane j owns sample j ----
      const int j = lane & (kM - 1);
      u64 z[kC / 2];
      {
        const u64* z0 = reinterpret_cast<const u64*>(&sm.partZ[0][j * kC]);
        const u64* z1 = reinterpret_cast<const u64*>(&sm.partZ[1][j * kC]);
        const u64* z2 = reinterpret_cast<const u64*>(&sm.partZ[2][j * kC]);
        const u64* z3 = reinterpret_cast<const u64*>(&sm.partZ[3][j * kC]);
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) z[c] = add2(add2(z0[c], z1[c]), add2(z2[c], z3[c]));
      }
      // column j of the Gram matrix: G[s][j], s < j; the warp that ran R for block k-1 has no share in it
      float Gj[kM - 1];
      {
        const int skip = (k + kWarps - 1) & (kWarps - 1);
        const int base = j * (j - 1) / 2;
#pragma unroll
        for (int s = 0; s < kM - 1; ++s) {
          const int idx = s < j ? base + s : 0;
          float acc = 1.f;   // the bias "pixel"
#pragma unroll
          for (int w = 0; w < kWarps; ++w)
            if (w != skip) acc += sm.partG[k & 1][w][idx];
          Gj[s] = acc;
        }
      }
      const int y = sm.ys[slot][j];
      u64 oh[kC / 2];
      {
        const ulonglong2* q = reinterpret_cast<const ulonglong2*>(&sm.onehot[((unsigned)y < (unsigned)kC) ? y : 0][0]);
        const ulonglong2 o0 = q[0], o1 = q[1], o2 = q[2];
        oh[0] = o0.x; oh[1] = o0.y; oh[2] = o1.x; oh[3] = o1.y; oh[4] = o2.x;
      }
#pragma unroll
      for (int s = 0; s < kM; ++s) {
        if ((uint32_t)s < nv) {      // uniform
          float zf[kC];
#pragma unroll
          for (int c = 0; c < kC / 2; ++c) unpack2(z[c], zf[2 * c], zf[2 * c + 1]);
          const float m = fmaxf(fmaxf(fmaxf(fmaxf(zf[0], zf[1]), fmaxf(zf[2], zf[3])), fmaxf(fmaxf(zf[4], zf[5]), fmaxf(zf[6], zf[7]))),
                                fmaxf(zf[8], zf[9]));
          const float nms = -m * kLog2e;
          const u64 nms2 = pack2(nms, nms);
          u64 e2[kC / 2];
#pragma unroll
          for (int c = 0; c < kC / 2; ++c) {
            float lo, hi;
            unpack2(fma2(z[c], log2e2, nms2), lo, hi);
            e2[c] = pack2(ex2(lo), ex2(hi));
          }
          float slo, shi;
          unpack2(add2(add2(add2(e2[0], e2[1]), add2(e2[2], e2[3])), e2[4]), slo, shi);
          const float inv = rcp(slo + shi);
          const u64 inv2 = pack2(inv, inv);
          u64 d2[kC / 2], nd2[kC / 2];
#pragma unroll
          for (int c = 0; c < kC / 2; ++c) {
            d2[c] = fma2(e2[c], inv2, oh[c]);
            nd2[c] = mul2(d2[c], neta2);
          }
          if (lane == s) {
            ulonglong2* dq = reinterpret_cast<ulonglong2*>(&sm.dbuf[s][0]);
            dq[0] = make_ulonglong2(d2[0], d2[1]);
            dq[1] = make_ulonglong2(d2[2], d2[3]);
            dq[2] = make_ulonglong2(d2[4], 0ull);
            dq[3] = make_ulonglong2(nd2[0], nd2[1]);
            dq[4] = make_ulonglong2(nd2[2], nd2[3]);
            dq[5] = make_ulonglong2(nd2[4], 0ull);
          }
          if (s + 1 < kM) {
            const float gs = Gj[s < kM - 1 ? s : 0];
            const u64 g2 = j > s ? pack2(gs, gs) : 0ull;   // earlier samples are done: no correction
#pragma unroll
            for (int c = 0; c < kC / 2; ++c) {
              const u64 nds = __shfl_sync(0xffffffffu, nd2[c], s);
              z[c] = fma2(nds, g2, z[c]);
            }
          }
        }
      }
    } else {
      const int rank = ((warp - rwarp) & (kWarps - 1)) - 1;   // 0..2 among the three other warps
      if (rank == 0 && k + 2 < nblk) produce(k + 2);          // its slot held block k-1: free since barrier A
      if (k + 1 < nblk) {
        ok = mbar_wait(&sm.full[(k + 1) % kSlots], ((k + 1) / kSlots) & 1) && ok;
        gram_partial(k + 1, rank);
      }
    }
    __syncthreads();   // barrier B: delta of the block is in shared memory

    // ---- P3: W -= eta * delta_t x_t^T, U += delta_t x_t^T ----
    auto apply_sample = [&](int s) {
      const ulonglong2* dq = reinterpret_cast<const ulonglong2*>(&sm.dbuf[s][0]);
      const ulonglong2 q0 = dq[0], q1 = dq[1], q2 = dq[2], q3 = dq[3], q4 = dq[4], q5 = dq[5];
      const u64 d2[kC / 2] = {q0.x, q0.y, q1.x, q1.y, q2.x};
      const u64 nd2[kC / 2] = {q3.x, q3.y, q4.x, q4.y, q5.x};
#pragma unroll
      for (int a = 0; a < kPx; ++a) {
        const float x = xslot[s * rs + a];
        const u64 xs = pack2(x, x);
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) {
          U2[a][c] = fma2(xs, d2[c], U2[a][c]);
          W2[a][c] = fma2(xs, nd2[c], W2[a][c]);
        }
      }
    };
    if (nv == kM) {
#pragma unroll
      for (int s = 0; s < kM; ++s) apply_sample(s);
    } else {
      for (uint32_t s = 0; s < nv; ++s) apply_sample((int)s);
    }
  }

  if (timed_out) {
    // A block of rows never arrived.  Flag it, give the copies still in flight a
    // bounded chance to land (their target is this CTA's shared memory), and leave.
    if (threadIdx.x == 0) {
      if (p.status) atomicOr(p.status, 1u);
      for (uint32_t j = timeout_at; j < nblk && j < timeout_at + 2; ++j) mbar_wait(&sm.full[j % kSlots], (j / kSlots) & 1);
    }
    return;
  }

  // ---- event trigger: h reached s_{i,c}; publish U_i (and the end model) ----
  if (owns) {
    float2* dU = reinterpret_cast<float2*>(p.U + (size_t)t.seq * p.stride + poff);
    float2* dW = p.w_end ? reinterpret_cast<float2*>(p.w_end + (size_t)t.seq * p.stride + poff) : nullptr;
#pragma unroll
    for (int a = 0; a < kPx; ++a)
#pragma unroll
      for (int c = 0; c < kC / 2; ++c) {
        if (active || a == 0) {
          float lo, hi;
          unpack2(U2[a][c], lo, hi);
          dU[a * (kC / 2) + c] = make_float2(lo, hi);
          if (dW) {
            unpack2(W2[a][c], lo, hi);
            dW[a * (kC / 2) + c] = make_float2(lo, hi);
          }
        }
      }
  }
  if (threadIdx.x == 0) {
    TriggerRec rec;
    rec.client = t.client; rec.round = t.round; rec.samples_done = n; rec.flags = 1;
    p.trig[t.seq] = rec;
  }
}

// Exercises the give-up path of the bounded wait without any faulty hardware:
// an mbarrier that nothing ever arrives on is polled `max_polls` times, then the
// CTA flags `status` exactly as a round kernel does and returns normally.
__global__ void wait_probe_kernel(uint32_t* status, uint32_t max_polls) {
  __shared__ __align__(8) uint64_t never;
  if (threadIdx.x == 0) {
    mbar_init(&never, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool landed = mbar_wait_limit(&never, 0, max_polls);
  if (__syncthreads_or(!landed) && threadIdx.x == 0) atomicOr(status, 1u);
}

}  // namespace

cudaError_t launch_wait_probe(uint32_t* status, uint32_t max_polls, cudaStream_t s) {
  wait_probe_kernel<<<1, 32, 0, s>>>(status, max_polls);
  return cudaGetLastError();
}

cudaError_t launch_lr_rounds(const RoundLaunch& p, cudaStream_t s) {
  if (p.n_tasks == 0) return cudaSuccess;
  if (p.l2 == 0.f) {
    // more than 48 KB of shared memory has to be asked for once per device
    static bool opted_in[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !opted_in[dev]) {
      e = cudaFuncSetAttribute(lr_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BlkSmem));
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) opted_in[dev] = true;
    }
    lr_block_kernel<<<p.n_tasks, kThreads, sizeof(BlkSmem), s>>>(p);
    return cudaGetLastError();
  }
  // lambda != 0 couples the steps of a block through the decay of W: step by step.
  // Enough round-tasks to put two CTAs on every SM: trade latency for instruction count.
  const bool shared = p.n_tasks >= 2 * 148;
  if (shared) lr_round_kernel<true, true><<<p.n_tasks, kThreads, 0, s>>>(p);
  else lr_round_kernel<true, false><<<p.n_tasks, kThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace aet
