// Local-SGD round of one client for softmax regression 784 -> 10, batch 1.
//
// Algorithm 3, MainComputeNode, inner loop: "sample xi; g = grad f(w_c, xi);
// w_c -= eta_i * g; U_i += g; h++" repeated s_{i,c} times, then the tuple
// (c, U_i, i) is sent.  One CTA runs one round-task; the client's model and
// the running update sum stay in registers for the whole round and only the
// sampled rows stream in from HBM.
//
// Two kernels live here.  lr_round_kernel takes the steps one by one and serves
// lambda != 0; lr_block_kernel (further down, with its own description) takes
// eight steps per block and serves lambda = 0, in a 4-warp instance for crowded
// launches and an 8-warp instance for launches with an SM per round-task.
//
// lr_round_kernel.  Work split: 4 warps (one per SM sub-partition), 98 threads own 8 consecutive
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
#include "lr_common.cuh"

namespace aet {
namespace {

using namespace lr;

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
  if (!debug_task_ok(p, t)) return;   // debug checks only: rows and slots in range, else flag and skip
  if (t.n_samples == 0) { publish_empty_round(p, t, kD * kC + kC); return; }
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
      const float* us = p.U + (size_t)ref.row * p.stride;
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
    float2* dU = reinterpret_cast<float2*>(p.U + (size_t)t.u_row * p.stride + off);
    float2* dW = p.w_end ? reinterpret_cast<float2*>(p.w_end + (size_t)t.u_row * p.stride + off) : nullptr;
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
// because W_t = W - eta * sum_{s<t} delta_s x_s^T.  And since eta is constant
// within a round and lambda = 0, W = W_start - eta * U at every block boundary,
// so only U is updated sample by sample.  Per block:
//   P1  W = W_start - eta U (registers, one FMA per parameter), Z0 = W X (every
//       thread: 14 pixels x 5 classes x kM samples), summed over the CTA by a
//       transposing shuffle butterfly and 4 per-warp partials in shared memory;
//   R   one warp (rotating) walks the kM samples: lane t owns sample t, takes the
//       softmax of its corrected logits and hands -eta*delta_t to the later
//       samples' lanes by shuffle; delta goes to shared memory; meanwhile the
//       other three warps compute the Gram matrix of the NEXT block (it does not
//       depend on W) and one of them issues the bulk copies of the block after it;
//   P3  U += delta_t x_t^T for the block's samples.
// The result equals the step-by-step recursion up to fp32 rounding order.  One
// barrier pair per kM samples instead of one per sample, and the latency-bound
// softmax chain of one block overlaps the FMA phases of the CTA sharing the SM.
// All FMAs here are scalar: on this part fma.rn.f32x2 with three distinct
// register pairs issues every ~3 cycles, a scalar fma every cycle.
//
// Work split: lane = 2 * (pixel group) + (class half).  4 warps x 14 groups x
// 14 consecutive pixels = 784; lanes 28, 29 of the last warp carry the bias as
// an always-1 pixel.  W_start and U stay in registers (2 x 70).  Rows arrive by
// cp.async.bulk into a ring of 3 blocks, issued two blocks ahead; every
// mbarrier wait is bounded.
constexpr int kSlots = 3;              // blocks of rows in shared memory
constexpr int kPx = 14, kPl = 14;      // pixels per thread, pixel groups per warp
static_assert(kPl * kWarps * kPx == kD, "pixel split");
static_assert(kM == 8, "lane-per-sample recurrence and butterfly widths assume 8");

struct __align__(128) BlkSmem {
  float rows[kSlots][kM][kD];
  float partZ[kWarps][kM * kC];       // per-warp totals of Z0, index t*10 + c
  float partG[2][kWarps][32];         // per-warp totals of the Gram pairs, double-buffered by block parity
  float dbuf[kM][16];                 // delta_t: classes 0..4 at [0..4], 5..9 at [8..12]
  float consts[32];                   // [0..13] = 1,0,...,0 (bias lanes' "row"); [16..29] = 0 (idle lanes)
  int ys[kSlots][kM];
  uint64_t full[kSlots];
  uint64_t staged;                    // completion of a bulk copy into stage[]
  float stage[kStageFloats];          // one model row on its way in (snapshot, in-flight sums) or out (U, end model)
};

// kDed: two more warps that own no pixels.  Warp 4 runs R and hands each delta_t to the four
// pixel warps through a hardware named barrier of its own, so that P3 streams under R instead
// of following it; warps 5 and 6 compute the Gram matrix of the next block, warp 7 issues the row
// copies (fetching their labels stalls it for an HBM round trip).  255 registers x 256 threads leave room for one such CTA per SM: the variant for launches
// with at most one round-task per SM, where a round-task's latency is all that counts.
template <bool kDed>
__global__ void __launch_bounds__(kDed ? 2 * kThreads : kThreads, kDed ? 1 : 2) lr_block_kernel(RoundLaunch p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  BlkSmem& sm = *reinterpret_cast<BlkSmem*>(smem_raw);
  constexpr int kHand = kThreads + 32;                    // threads meeting at a delta hand-over: pixel warps + R warp
  constexpr int kGramRanks = kDed ? 2 : kWarps - 1;       // warps sharing the Gram matrix of a block

  const TaskDesc t = p.tasks[p.task_begin + blockIdx.x];
  if (!debug_task_ok(p, t)) return;   // debug checks only: rows and slots in range, else flag and skip
  if (t.n_samples == 0) {   // this grid may run under the tail of the aggregation before it: wait before writing
    asm volatile("griddepcontrol.wait;" ::: "memory");
    publish_empty_round(p, t, kParams);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool rw = kDed && warp >= kWarps;            // the warps without pixels: R (warp 4), Gram and row copies (warp 5)
  const bool gw = kDed && (warp == kWarps + 1 || warp == kWarps + 2);   // warps 5 and 6
  const int cg = lane & 1, pl = lane >> 1;
  const bool active = !rw && pl < kPl;
  const bool is_bias = warp == kWarps - 1 && pl == kPl;
  const int pg = rw ? 0 : warp * kPl + (active ? pl : 0);     // pixel group: pixels 14 pg .. 14 pg + 13

  const ClientData cd = p.clients[t.client];
  const uint64_t key = p.sample_keys[t.client];
  const float* xrows = reinterpret_cast<const float*>(cd.x);
  const uint32_t n = t.n_samples;
  const uint32_t nblk = (n + kM - 1) / kM;
  const float neta = -t.eta;

  if (threadIdx.x == 0) {
#pragma unroll
    for (int s = 0; s < kSlots; ++s) mbar_init(&sm.full[s], 1);
    mbar_init(&sm.staged, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) sm.consts[threadIdx.x] = threadIdx.x == 0 ? 1.f : 0.f;
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
  // ---- start model: server snapshot minus own update sums still in flight ----
  // Ws[a][c] = W[14 pg + a][5 cg + c]; the bias lanes hold b[5 cg + c] in row 0.
  // A thread's 70 parameters are 20-byte pieces 40 bytes apart: each row comes in
  // as one bulk copy and the threads pick their pieces out of shared memory.
  float Ws[kPx][kCh], U[kPx][kCh];
  const bool owns = active || is_bias;
  const size_t poff = (is_bias ? (size_t)kD * kC : (size_t)pg * (kPx * kC)) + (size_t)cg * kCh;
  const bool whole_rows = p.stride == (size_t)kStageFloats;   // rows as this kernel stages them
  bool ok = true;
  {
#pragma unroll
    for (int a = 0; a < kPx; ++a)
#pragma unroll
      for (int c = 0; c < kCh; ++c) { Ws[a][c] = 0.f; U[a][c] = 0.f; }
    // Everything above reads only what earlier, finished grids and the host wrote.  The snapshot
    // is written by the aggregation kernel launched just before this grid, which may still be
    // running when this grid was launched with programmatic stream serialisation.
    if (warp == 0) {   // the first two blocks of rows
      produce(0);
      if (nblk > 1) produce(1);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (uint32_t f = 0; f <= t.inflight_cnt; ++f) {   // f = 0: the snapshot, then the sums in flight
      const float* row;
      float scale;
      if (f == 0) {
        row = p.snaps + (size_t)t.snap_slot * p.stride;
        scale = 1.f;
      } else {
        const InflightRef ref = p.inflight[t.inflight_off + f - 1];
        row = p.U + (size_t)ref.row * p.stride;
        scale = -ref.eta;
      }
      if (whole_rows) {
        if (f) __syncthreads();   // everybody has taken the previous row out of stage[]
        if (threadIdx.x == 0) {
          mbar_expect_tx(&sm.staged, kStageFloats * sizeof(float));
          bulk_load(sm.stage, row, kStageFloats * sizeof(float), &sm.staged);
        }
      }
      if (whole_rows) {
        ok = mbar_wait(&sm.staged, f & 1) && ok;
        row = sm.stage;
      }
#pragma unroll
      for (int a = 0; a < kPx; ++a)
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
          const bool live = active || (is_bias && a == 0);
          const float v = live ? (whole_rows ? row[poff + a * kC + c] : __ldg(row + poff + a * kC + c)) : 0.f;
          Ws[a][c] = fmaf(scale, v, Ws[a][c]);
        }
    }
  }

  // Where this thread reads "its pixels" of sample (slot, t): pixel-owning lanes
  // from the row, the bias lanes from {1,0,...}, idle lanes from zeros (row stride 0).
  const float* xbase = active ? &sm.rows[0][0][pg * kPx] : (is_bias ? &sm.consts[0] : &sm.consts[16]);
  const int rs = active ? kD : 0;

  // where the lane's butterfly totals go
  static_assert(BflyDims<kM * kCh>::n4 == 3 && BflyDims<kPairs>::n5 == 1, "butterfly widths");
  int zidx[3];
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const int v = bfly_index4<kM * kCh>(lane, i);       // v = s * 5 + c
    zidx[i] = v < 0 ? -1 : (v / kCh) * kC + cg * kCh + (v % kCh);
  }
  const int gidx = bfly_index5<kPairs>(lane, 0);

  // Gram pairs of block kb over this warp's share of the pixels (rank r of 3).
  auto gram_partial = [&](uint32_t kb, int r) {
    const float* rb = &sm.rows[kb % kSlots][0][0];
    float gacc[kPairs];
#pragma unroll
    for (int i = 0; i < kPairs; ++i) gacc[i] = 0.f;
#pragma unroll 2
    for (int chunk = r; chunk * 32 < kD; chunk += kGramRanks) {
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
    bfly_reduce5<kPairs>(gacc, o, lane);
    if (gidx >= 0) sm.partG[kb & 1][kDed ? r : warp][gidx] = o[0];
  };

  bool timed_out = false;
  uint32_t timeout_at = 0;

  // Gram matrix of block 0: warps 0..2 (the rotation below treats warp 3 as busy before block 0),
  // or the Gram warp alone
  if (kDed ? gw : warp != kWarps - 1) {
    ok = mbar_wait(&sm.full[0], 0) && ok;
    gram_partial(0, kDed ? warp - (kWarps + 1) : warp);
  }

  for (uint32_t k = 0; k < nblk; ++k) {
    const int slot = k % kSlots;
    const uint32_t nv = min((uint32_t)kM, n - k * kM);
    ok = mbar_wait(&sm.full[slot], (k / kSlots) & 1) && ok;
    const float* xslot = xbase + (size_t)slot * kM * rs;

    // ---- P1: W = W_start - eta U; this thread's share of Z0 = W X ----
    if (!rw) {
      float acc[kM][kCh];
#pragma unroll
      for (int a2 = 0; a2 < kPx / 2; ++a2) {
        float w0[kCh], w1[kCh];
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
          w0[c] = fmaf(neta, U[2 * a2][c], Ws[2 * a2][c]);
          w1[c] = fmaf(neta, U[2 * a2 + 1][c], Ws[2 * a2 + 1][c]);
        }
#pragma unroll
        for (int s = 0; s < kM; ++s) {
          const float2 x = *reinterpret_cast<const float2*>(xslot + s * rs + 2 * a2);
#pragma unroll
          for (int c = 0; c < kCh; ++c) {
            acc[s][c] = a2 == 0 ? x.x * w0[c] : fmaf(x.x, w0[c], acc[s][c]);
            acc[s][c] = fmaf(x.y, w1[c], acc[s][c]);
          }
        }
      }
      float v[kM * kCh];
#pragma unroll
      for (int s = 0; s < kM; ++s)
#pragma unroll
        for (int c = 0; c < kCh; ++c) v[s * kCh + c] = acc[s][c];
      float o[3];
      bfly_reduce4<kM * kCh>(v, o, lane);
#pragma unroll
      for (int i = 0; i < 3; ++i)
        if (zidx[i] >= 0) sm.partZ[warp][zidx[i]] = o[i];
    }
    // barrier A: partials visible, rows of block k-1 no longer read by anyone; it
    // also carries the verdict of the bounded waits so that all threads leave together
    if (__syncthreads_or(!ok)) { timed_out = true; timeout_at = k; break; }

    const int rwarp = kDed ? kWarps : (int)(k & (kWarps - 1));
    if (warp == rwarp) {
      // ---- R: the block's kM dependent softmax steps, lane j owns sample j ----
      const int j = lane & (kM - 1);
      float z[kC];
      {
        const float2* z0 = reinterpret_cast<const float2*>(&sm.partZ[0][j * kC]);
        const float2* z1 = reinterpret_cast<const float2*>(&sm.partZ[1][j * kC]);
        const float2* z2 = reinterpret_cast<const float2*>(&sm.partZ[2][j * kC]);
        const float2* z3 = reinterpret_cast<const float2*>(&sm.partZ[3][j * kC]);
#pragma unroll
        for (int c = 0; c < kC / 2; ++c) {
          const float2 a0 = z0[c], a1 = z1[c], a2 = z2[c], a3 = z3[c];
          z[2 * c] = (a0.x + a1.x) + (a2.x + a3.x);
          z[2 * c + 1] = (a0.y + a1.y) + (a2.y + a3.y);
        }
      }
      // column j of the Gram matrix, one entry per step: -eta * G[s][j] for s < j, 0 for
      // the others (a finished sample takes no correction); the warp that ran R for block
      // k-1 has no share in the Gram partials.  Loaded one step ahead of its use.
      const int skip = kDed ? kWarps : (int)((k + kWarps - 1) & (kWarps - 1));
      const float* g0 = sm.partG[k & 1][skip == 0 ? 1 : 0];
      const float* g1 = sm.partG[k & 1][skip <= 1 ? 2 : 1];
      const float* g2 = sm.partG[k & 1][skip <= 2 ? 3 : 2];
      const int gbase = j * (j - 1) / 2;
      auto corr = [&](int s) -> float {
        const int idx = s < j ? gbase + s : 0;
        const float gsum = kDed ? (1.f + g0[idx]) + g1[idx] : (1.f + g0[idx]) + (g1[idx] + g2[idx]);   // 1 = the bias "pixel"
        return s < j ? gsum * neta : 0.f;
      };
      const int y = sm.ys[slot][j];
      float oh[kC];
#pragma unroll
      for (int c = 0; c < kC; ++c) oh[c] = c == y ? -1.f : 0.f;
      float gs = corr(0);
      // The loop stays rolled: the whole per-block body has to fit the instruction cache.
#pragma unroll 1
      for (int s = 0; s < (int)nv; ++s) {
        const float gnext = corr(s + 1);
        const float m = fmaxf(fmaxf(fmaxf(fmaxf(z[0], z[1]), fmaxf(z[2], z[3])), fmaxf(fmaxf(z[4], z[5]), fmaxf(z[6], z[7]))),
                              fmaxf(z[8], z[9]));
        const float nms = -m * kLog2e;
        float e[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) e[c] = ex2(fmaf(z[c], kLog2e, nms));
        const float sum = (((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]))) + (e[8] + e[9]);
        const float inv = rcp(sum);
        float d[kC];
#pragma unroll
        for (int c = 0; c < kC; ++c) d[c] = fmaf(e[c], inv, oh[c]);
        if (lane == s) {
          float4* dq = reinterpret_cast<float4*>(&sm.dbuf[s][0]);
          dq[0] = make_float4(d[0], d[1], d[2], d[3]);
          dq[1] = make_float4(d[4], 0.f, 0.f, 0.f);
          dq[2] = make_float4(d[5], d[6], d[7], d[8]);
          dq[3] = make_float4(d[9], 0.f, 0.f, 0.f);
        }
        if (kDed) named_arrive(1 + s, kHand);   // delta_s is out: the pixel warps may apply it
#pragma unroll
        for (int c = 0; c < kC; ++c) z[c] = fmaf(__shfl_sync(0xffffffffu, d[c], s), gs, z[c]);
        gs = gnext;
      }
    } else {
      // 0..2 among the three other warps; kDed: the Gram warp alone does this part
      const int rank = kDed ? warp - (kWarps + 1) : ((warp - rwarp) & (kWarps - 1)) - 1;
      const bool producer = kDed ? warp == kWarps + 3 : rank == 0;
      // block k+2's slot held block k-1: free since barrier A.  The copies' labels take an HBM round
      // trip, so the Gram warps (whose result R needs at the next barrier) fetch after their share.
      if (!kDed && producer && k + 2 < nblk) produce(k + 2);
      if ((!kDed || gw) && k + 1 < nblk) {
        ok = mbar_wait(&sm.full[(k + 1) % kSlots], ((k + 1) / kSlots) & 1) && ok;
        gram_partial(k + 1, rank);
      }
      if (kDed && producer && k + 2 < nblk) produce(k + 2);
    }
    if (!kDed) __syncthreads();   // barrier B: delta of the block is in shared memory

    // ---- P3: U += delta_t x_t^T (two samples per trip: the loop has to stay small, see R) ----
    if (!rw && !kDed) {
#pragma unroll 2
      for (int s = 0; s < (int)nv; ++s) {
        const float4 dq = *reinterpret_cast<const float4*>(&sm.dbuf[s][cg * 8]);
        const float d[kCh] = {dq.x, dq.y, dq.z, dq.w, sm.dbuf[s][cg * 8 + 4]};
#pragma unroll
        for (int a2 = 0; a2 < kPx / 2; ++a2) {
          const float2 x = *reinterpret_cast<const float2*>(xslot + s * rs + 2 * a2);
#pragma unroll
          for (int c = 0; c < kCh; ++c) {
            U[2 * a2][c] = fmaf(x.x, d[c], U[2 * a2][c]);
            U[2 * a2 + 1][c] = fmaf(x.y, d[c], U[2 * a2 + 1][c]);
          }
        }
      }
    }
    if (!rw && kDed) {
      // streaming under R: a sample's pixels are fetched before the wait for its delta
      float2 x[kPx / 2];
#pragma unroll
      for (int a2 = 0; a2 < kPx / 2; ++a2) x[a2] = *reinterpret_cast<const float2*>(xslot + 2 * a2);
#pragma unroll 1
      for (int s = 0; s < (int)nv; ++s) {
        named_sync(1 + s, kHand);   // delta_s has been written
        const float4 dq = *reinterpret_cast<const float4*>(&sm.dbuf[s][cg * 8]);
        const float d[kCh] = {dq.x, dq.y, dq.z, dq.w, sm.dbuf[s][cg * 8 + 4]};
        float2 xn[kPx / 2];
        const int sn = s + 1 < kM ? s + 1 : s;
#pragma unroll
        for (int a2 = 0; a2 < kPx / 2; ++a2) xn[a2] = *reinterpret_cast<const float2*>(xslot + sn * rs + 2 * a2);
#pragma unroll
        for (int a2 = 0; a2 < kPx / 2; ++a2) {
#pragma unroll
          for (int c = 0; c < kCh; ++c) {
            U[2 * a2][c] = fmaf(x[a2].x, d[c], U[2 * a2][c]);
            U[2 * a2 + 1][c] = fmaf(x[a2].y, d[c], U[2 * a2 + 1][c]);
          }
          x[a2] = xn[a2];
        }
      }
    }
  }

  if (timed_out) {
    // A block of rows never arrived.  Flag it, give the copies still in flight a
    // bounded chance to land (their target is this CTA's shared memory), and leave.
    if (threadIdx.x == 0) {
      if (p.status) atomicOr(p.status, 1u);
      for (uint32_t j = timeout_at; j < nblk && j < timeout_at + 2; ++j) mbar_wait(&sm.full[j % kSlots], (j / kSlots) & 1);
      if (whole_rows) mbar_wait(&sm.staged, t.inflight_cnt & 1);   // the last row staged at the start
    }
    return;
  }

  // The aggregation kernel behind this grid in the stream may become resident from here on (it
  // touches nothing until this grid has finished and its writes are visible).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ---- event trigger: h reached s_{i,c}; publish U_i (and the end model W_start - eta U) ----
  for (int pass = 0; pass < (p.w_end ? 2 : 1); ++pass) {
    float* dst = (pass == 0 ? p.U : p.w_end) + (size_t)t.u_row * p.stride;
    float* out = whole_rows ? sm.stage : dst;
    if (whole_rows) {
      if (pass) __syncthreads();   // the previous row has left stage[]
      if (threadIdx.x < kStageFloats - kParams) sm.stage[kParams + threadIdx.x] = 0.f;   // the row's padding
    }
    if (owns) {
#pragma unroll
      for (int a = 0; a < kPx; ++a)
#pragma unroll
        for (int c = 0; c < kCh; ++c)
          if (active || a == 0) out[poff + a * kC + c] = pass == 0 ? U[a][c] : fmaf(neta, U[a][c], Ws[a][c]);
    }
    if (whole_rows) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads what the threads wrote
      __syncthreads();
      if (threadIdx.x == 0) bulk_store_and_wait(dst, sm.stage, kStageFloats * sizeof(float));
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
    static int sm_count[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool known = dev >= 0 && dev < 64;
    int sms = known ? sm_count[dev] : 0;
    if (!known || !opted_in[dev]) {
      e = cudaFuncSetAttribute(lr_block_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BlkSmem));
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(lr_block_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(BlkSmem));
      if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return e;
      if (known) { opted_in[dev] = true; sm_count[dev] = sms; }
    }
    // More round-tasks than SMs: the kernel that keeps the update sum in tensor memory.
    if ((p.n_tasks > (uint32_t)sms || p.crowded_hint) && lr_tc_eligible(p)) return launch_lr_tc_rounds(p, s);
    // At most one round-task per SM: the variant with a warp of its own for the softmax recurrence.
    const bool dedicated = p.n_tasks <= (uint32_t)sms;
    // Programmatic stream serialisation: the grid may start while the kernel before it in the
    // stream (the aggregation of the previous wave) is still running; lr_block_kernel waits
    // (griddepcontrol.wait) before it reads anything that kernel writes.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.n_tasks, 1, 1);
    cfg.blockDim = dim3(dedicated ? 2 * kThreads : kThreads, 1, 1);
    cfg.dynamicSmemBytes = sizeof(BlkSmem);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return dedicated ? cudaLaunchKernelEx(&cfg, lr_block_kernel<true>, p) : cudaLaunchKernelEx(&cfg, lr_block_kernel<false>, p);
  }
  // lambda != 0 couples the steps of a block through the decay of W: step by step.
  // Enough round-tasks to put two CTAs on every SM: trade latency for instruction count.
  const bool shared = p.n_tasks >= 2 * 148;
  if (shared) lr_round_kernel<true, true><<<p.n_tasks, kThreads, 0, s>>>(p);
  else lr_round_kernel<true, false><<<p.n_tasks, kThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace aet
