// Local-SGD round of one client for a small convolutional classifier (the LeNet shape the paper
// trains on its 28x28 sets; Appendix, "Objective function"):
//   conv 5x5 valid (c_in -> c1) + bias, ReLU, 2x2 average pooling,
//   conv 5x5 valid (c1 -> c2) + bias, ReLU, 2x2 average pooling, flatten [c2][y][x],
//   dense f1, ReLU, dense f2, ReLU, dense classes, softmax cross-entropy.
// Algorithm 3, MainComputeNode, inner loop with xi a minibatch: g = mean gradient (+ lambda W on
// weight tensors), w_c -= eta_i g, U_i += g, repeated s_{i,c} / B times; then (c, U_i, i) is sent.
//
// A cluster of up to 8 CTAs of 512 threads per round-task, the minibatch split over the CTAs.  Every
// CTA keeps the client's whole model (44,426 parameters for the 28x28 shape, 174 KB) in shared memory
// from the start of the round to its trigger and runs the forward and backward pass of its own
// samples (activations in global scratch, L2-resident) against the same, old weights; each
// parameter's gradient over the CTA's samples goes to a per-CTA row of global scratch.  After a
// cluster barrier every CTA owns a slice of the parameters: it adds the slice over the CTAs' rows in
// rank order (no atomics, identical from run to run), applies w -= eta g and U += g, and writes the
// new weights into all the CTAs' copies through distributed shared memory; a second barrier ends the
// iteration.  With one CTA (a launch too full for clusters, or a minibatch of one) the same code runs
// with a cluster of one.
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"

namespace aet {
namespace {

constexpr int kCnnThreads = 512;
constexpr int kK = 5;   // kernel side of both convolutions
constexpr int kMaxCl = 8;   // CTAs per round-task at most

struct CnnDims {
  int side, cin, c1, c2, f1, f2, ncls, s1, p1, s2, p2, flat;
  int oW1, ob1, oW2, ob2, oF1, obF1, oF2, obF2, oF3, obF3, P, Ppad;
  // per-minibatch activation scratch (floats), offsets for batch size B
  int a1, q1, a2, q2, h1, h2, z3, dz3, dh2, dh1, dq2, dq1, total;
};

__host__ __device__ constexpr CnnDims make_cnn_dims(const CnnShape& s) {
  CnnDims d{};
  d.side = (int)s.dims[0]; d.cin = (int)s.dims[1]; d.c1 = (int)s.dims[2]; d.c2 = (int)s.dims[3];
  d.f1 = (int)s.dims[4]; d.f2 = (int)s.dims[5]; d.ncls = (int)s.dims[6];
  d.s1 = d.side - kK + 1; d.p1 = d.s1 / 2; d.s2 = d.p1 - kK + 1; d.p2 = d.s2 / 2;
  d.flat = d.c2 * d.p2 * d.p2;
  int o = 0;
  d.oW1 = o; o += d.c1 * d.cin * kK * kK; d.ob1 = o; o += d.c1;
  d.oW2 = o; o += d.c2 * d.c1 * kK * kK; d.ob2 = o; o += d.c2;
  d.oF1 = o; o += d.flat * d.f1; d.obF1 = o; o += d.f1;
  d.oF2 = o; o += d.f1 * d.f2; d.obF2 = o; o += d.f2;
  d.oF3 = o; o += d.f2 * d.ncls; d.obF3 = o; o += d.ncls;
  d.P = o;
  d.Ppad = (o + 31) & ~31;
  const int B = (int)s.batch;
  int a = 0;
  d.a1 = a; a += B * d.c1 * d.s1 * d.s1;
  d.q1 = a; a += B * d.c1 * d.p1 * d.p1;
  d.a2 = a; a += B * d.c2 * d.s2 * d.s2;
  d.q2 = a; a += B * d.flat;
  d.h1 = a; a += B * d.f1;
  d.h2 = a; a += B * d.f2;
  d.z3 = a; a += B * d.ncls;
  d.dz3 = a; a += B * d.ncls;
  d.dh2 = a; a += B * d.f2;
  d.dh1 = a; a += B * d.f1;
  d.dq2 = a; a += B * d.flat;
  d.dq1 = a; a += B * d.c1 * d.p1 * d.p1;
  d.total = (a + 31) & ~31;
  return d;
}

// Valid 5x5 correlation + bias + ReLU + 2x2 average pooling of one stage, for samples [b0, b0 + nb).
// One work item = one pooled output: its four pre-pooling outputs share a 6x6 input patch per plane.
template <class InAt>
__device__ __forceinline__ void conv_stage(int b0, int nb, int cin, int cout, int sin, int sout, const float* W, const float* bias,
                                           InAt in_at, float* a_out, float* q_out, int tid) {
  const int pout = sout / 2;
  const int items = nb * cout * pout * pout;
  for (int e = tid; e < items; e += kCnnThreads) {
    const int px = e % pout, py = (e / pout) % pout, c = (e / (pout * pout)) % cout, b = b0 + e / (pout * pout * cout);
    float z00 = bias[c], z01 = z00, z10 = z00, z11 = z00;
    for (int ci = 0; ci < cin; ++ci) {
      float patch[6][6];
#pragma unroll
      for (int r = 0; r < 6; ++r)
#pragma unroll
        for (int q = 0; q < 6; ++q) patch[r][q] = in_at(b, ci, 2 * py + r, 2 * px + q);
      const float* wk = W + (c * cin + ci) * (kK * kK);
#pragma unroll
      for (int dy = 0; dy < kK; ++dy)
#pragma unroll
        for (int dx = 0; dx < kK; ++dx) {
          const float wv = wk[dy * kK + dx];
          z00 = fmaf(wv, patch[dy][dx], z00);
          z01 = fmaf(wv, patch[dy][dx + 1], z01);
          z10 = fmaf(wv, patch[dy + 1][dx], z10);
          z11 = fmaf(wv, patch[dy + 1][dx + 1], z11);
        }
    }
    z00 = fmaxf(z00, 0.f); z01 = fmaxf(z01, 0.f); z10 = fmaxf(z10, 0.f); z11 = fmaxf(z11, 0.f);
    float* ao = a_out + ((size_t)(b * cout + c) * sout + 2 * py) * sout + 2 * px;
    ao[0] = z00; ao[1] = z01; ao[sout] = z10; ao[sout + 1] = z11;
    q_out[((size_t)(b * cout + c) * pout + py) * pout + px] = 0.25f * ((z00 + z01) + (z10 + z11));
  }
}

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// floats of per-sample activations that may live in shared memory (everything but the first convolution's maps)
__host__ __device__ constexpr int cnn_small_acts(const CnnDims& d) {
  return 2 * d.c1 * d.p1 * d.p1 + d.c2 * d.s2 * d.s2 + 2 * d.flat + 2 * d.f1 + 2 * d.f2 + 2 * d.ncls;
}

// The shape the paper trains on its 28x28 sets, minibatch 16 on a cluster of 8: with every extent a compile-time
// constant the index arithmetic folds and the short loops unroll (the general instance executes 34 K instructions
// per thread and iteration, most of them divisions by run-time extents and 64-bit address arithmetic).
constexpr CnnShape kLeNetShape = {{28, 1, 6, 16, 120, 84, 10, 0}, 16};

// kFixed: kLeNetShape on a cluster of 8, rows and activations staged; otherwise everything is read from the launch.
template <bool kFixed>
__global__ void __launch_bounds__(kCnnThreads, 1) cnn_round_kernel(CnnLaunch p) {
  extern __shared__ __align__(16) float smem[];
  const int CL = kFixed ? kMaxCl : (int)cluster_size(), rank = (int)cluster_rank();
  const int task = blockIdx.x / CL;
  const TaskDesc t = p.r.tasks[p.r.task_begin + task];
  if (!debug_task_ok(p.r, t)) return;   // debug checks only: rows and slots in range, else flag and skip (the whole cluster alike)
  constexpr CnnDims kFixedDims = make_cnn_dims(kLeNetShape);
  const CnnDims D = kFixed ? kFixedDims : make_cnn_dims(p.shape);
  const int B = kFixed ? (int)kLeNetShape.batch : (int)p.shape.batch;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float* w = smem;                                     // the client's model, whole round, one copy per CTA
  int* idx = reinterpret_cast<int*>(smem + ((D.P + 3) & ~3));
  int* ylab = idx + B;

  const ClientData cd = p.r.clients[t.client];
  const float* xrows = reinterpret_cast<const float*>(cd.x);
  const uint64_t key = p.r.sample_keys[t.client];
  const float eta = t.eta, lambda = p.r.l2, invB = 1.f / (float)B;
  const int rowlen = D.cin * D.side * D.side;
  float* act = p.act + (size_t)task * p.act_stride;
  float* Urow = p.r.U + (size_t)t.u_row * p.r.stride;
  // this CTA's samples of the minibatch, its row of gradient partials, its slice of the parameters
  const int per = (B + CL - 1) / CL, nact = (B + per - 1) / per;
  const int b0 = kFixed ? rank * per : min(B, rank * per), nb = kFixed ? per : min(B, b0 + per) - b0;   // kFixed: 16 = 8 x 2
  float* G = act + D.total + (size_t)rank * D.Ppad;
  const int slice = (D.P + CL - 1) / CL, k_lo = min(D.P, rank * slice), k_hi = min(D.P, k_lo + slice);
  // Where the launch found room, the CTA's minibatch rows and all its activations except the first convolution's
  // maps sit in shared memory behind the model (indexed by the sample's place in the minibatch all the same);
  // otherwise they stay in global scratch.
  const bool rows_staged = kFixed || p.stage_rows != 0, acts_staged = kFixed || p.stage_acts != 0;
  float* xs = reinterpret_cast<float*>(ylab + B);
  float* sa = xs + (rows_staged ? per * rowlen : 0);
  auto place = [&](int per_sample, int global_off) -> float* {
    if (!acts_staged) return act + global_off;
    float* r = sa - (ptrdiff_t)b0 * per_sample;
    sa += per * per_sample;
    return r;
  };
  const int n_q1 = D.c1 * D.p1 * D.p1, n_a2 = D.c2 * D.s2 * D.s2, n_a1 = D.c1 * D.s1 * D.s1;
  float* a1 = act + D.a1;
  float* q1 = place(n_q1, D.q1);
  float* a2 = place(n_a2, D.a2);
  float* q2 = place(D.flat, D.q2);
  float* h1 = place(D.f1, D.h1);
  float* h2 = place(D.f2, D.h2);
  float* z3 = place(D.ncls, D.z3);
  float* dz3 = place(D.ncls, D.dz3);
  float* dh2 = place(D.f2, D.dh2);
  float* dh1 = place(D.f1, D.dh1);
  float* dq2 = place(D.flat, D.dq2);
  float* dq1 = place(n_q1, D.dq1);

  // ---- start model: snapshot minus own update sums still in flight; U_i = 0 ----
  {
    const float* snap = p.r.snaps + (size_t)t.snap_slot * p.r.stride;
    // eight parameters per thread and trip, all loads of a trip before its first store (the stores to U could
    // alias the loads for all the compiler knows, which would leave one load in flight per thread)
    constexpr int kTrip = 8;
    for (int kb = tid; kb < D.P; kb += kTrip * kCnnThreads) {
      float v[kTrip];
#pragma unroll
      for (int q = 0; q < kTrip; ++q) v[q] = kb + q * kCnnThreads < D.P ? snap[kb + q * kCnnThreads] : 0.f;
      for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
        const InflightRef ref = p.r.inflight[t.inflight_off + f];
        const float* urow = p.r.U + (size_t)ref.row * p.r.stride;
        float u[kTrip];
#pragma unroll
        for (int q = 0; q < kTrip; ++q) u[q] = kb + q * kCnnThreads < D.P ? urow[kb + q * kCnnThreads] : 0.f;
#pragma unroll
        for (int q = 0; q < kTrip; ++q) v[q] = fmaf(-ref.eta, u[q], v[q]);
      }
#pragma unroll
      for (int q = 0; q < kTrip; ++q) {
        const int k = kb + q * kCnnThreads;
        if (k < D.P) {
          w[k] = v[q];
          if (k >= k_lo && k < k_hi) Urow[k] = 0.f;
        }
      }
    }
  }
  __syncthreads();

  for (uint32_t it = 0; it < t.steps; ++it) {
    if (tid < B) {
      const int id = (int)sample_index(draw(key, t.sample_ctr0 + (uint64_t)it * B + tid), cd.n);
      idx[tid] = id;
      ylab[tid] = __ldg(cd.y + id);
    }
    __syncthreads();
    if (rows_staged) {   // the rows are read 25 times over by the first convolution and its gradient: one coalesced copy first
      for (int e = tid; e < nb * rowlen; e += kCnnThreads) xs[e] = __ldg(xrows + (size_t)idx[b0 + e / rowlen] * rowlen + e % rowlen);
      __syncthreads();
    }
    // pixel (ci, y, x) of minibatch sample b (one of this CTA's)
    auto x_at = [&](int b, int ci, int y, int x) {
      const int at = (ci * D.side + y) * D.side + x;
      return rows_staged ? xs[(b - b0) * rowlen + at] : __ldg(xrows + (size_t)idx[b] * rowlen + at);
    };

    // ================= forward (own samples) =================
    conv_stage(b0, nb, D.cin, D.c1, D.side, D.s1, w + D.oW1, w + D.ob1, x_at, a1, q1, tid);
    __syncthreads();
    conv_stage(b0, nb, D.c1, D.c2, D.p1, D.s2, w + D.oW2, w + D.ob2,
               [&](int b, int ci, int y, int x) { return q1[((size_t)(b * D.c1 + ci) * D.p1 + y) * D.p1 + x]; }, a2, q2, tid);
    __syncthreads();
    auto dense_fwd = [&](const float* in, int K, int N, const float* Wl, const float* bl, float* out, bool relu) {
      for (int e = tid; e < nb * N; e += kCnnThreads) {
        const int j = e % N, b = b0 + e / N;
        float z0 = bl[j], z1 = 0.f, z2 = 0.f, z3v = 0.f;   // four chains: the operands come from shared memory with latency
        const float* a = in + (size_t)b * K;
        int k = 0;
        for (; k + 4 <= K; k += 4) {
          z0 = fmaf(a[k], Wl[k * N + j], z0);
          z1 = fmaf(a[k + 1], Wl[(k + 1) * N + j], z1);
          z2 = fmaf(a[k + 2], Wl[(k + 2) * N + j], z2);
          z3v = fmaf(a[k + 3], Wl[(k + 3) * N + j], z3v);
        }
        for (; k < K; ++k) z0 = fmaf(a[k], Wl[k * N + j], z0);
        const float z = (z0 + z1) + (z2 + z3v);
        out[(size_t)b * N + j] = relu ? fmaxf(z, 0.f) : z;
      }
    };
    dense_fwd(q2, D.flat, D.f1, w + D.oF1, w + D.obF1, h1, true);
    __syncthreads();
    dense_fwd(h1, D.f1, D.f2, w + D.oF2, w + D.obF2, h2, true);
    __syncthreads();
    dense_fwd(h2, D.f2, D.ncls, w + D.oF3, w + D.obF3, z3, false);
    __syncthreads();
    if (tid < nb) {   // softmax cross-entropy: dZ = (p - onehot) / B
      const int b = b0 + tid;
      const float* z = z3 + b * D.ncls;
      float m = -INFINITY;
      for (int j = 0; j < D.ncls; ++j) m = fmaxf(m, z[j]);
      float sum = 0.f;
      for (int j = 0; j < D.ncls; ++j) sum += __expf(z[j] - m);
      const float inv = 1.f / sum;
      const int y = ylab[b];
      for (int j = 0; j < D.ncls; ++j) dz3[b * D.ncls + j] = (__expf(z[j] - m) * inv - (j == y ? 1.f : 0.f)) * invB;
    }
    __syncthreads();

    // ================= backward (own samples, old weights throughout) =================
    constexpr int kW = kCnnThreads / 32, kGradW = 4;
    // Input gradient of a dense layer, gated by the ReLU of the layer below: dIn[b, i] = [in > 0] sum_j dOut[b, j] W[i, j].
    // Warps `wfirst`, `wfirst + wstep`, ... take the (sample, input) pairs in turn; lanes run along row i of W
    // (contiguous in shared memory) and meet in a shuffle tree.
    auto dense_din = [&](int wfirst, int wstep, const float* dout, int K, int N, const float* Wl, const float* in, float* din, bool gate) {
      for (int e = wfirst; e < nb * K; e += wstep) {
        const int i = e % K, b = b0 + e / K;
        const float* dz = dout + (size_t)b * N;
        const float* wr = Wl + (size_t)i * N;
        float s = 0.f;
        for (int j = lane; j < N; j += 32) s = fmaf(dz[j], wr[j], s);
#pragma unroll
        for (int m = 16; m; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
        const size_t at = (size_t)b * K + i;
        if (lane == 0) din[at] = (!gate || in[at] > 0.f) ? s : 0.f;
      }
    };
    // This CTA's share of the gradient of a dense layer: warps `wfirst`, `wfirst + wstep`, ... of the CTA take the
    // input rows in turn (row K is the bias), lanes run across the outputs - no index arithmetic per parameter.
    auto dense_grad = [&](int wfirst, int wstep, const float* in, const float* dout, int K, int N, int oW, int ob) {
      if (nb <= 4) {
        // few samples per CTA: a lane keeps its column of dOut in registers and walks the rows
        for (int j = lane; j < N; j += 32) {
          float d[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) d[q] = q < nb ? dout[(size_t)(b0 + q) * N + j] : 0.f;
          for (int i = wfirst; i < K; i += wstep) {
            float g = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (q < nb) g = fmaf(in[(size_t)(b0 + q) * K + i], d[q], g);
            G[oW + i * N + j] = g;
          }
          if (wfirst == K % wstep) G[ob + j] = ((d[0] + d[1]) + d[2]) + d[3];   // the bias row, by the warp whose turn it would be
        }
        return;
      }
      for (int i = wfirst; i <= K; i += wstep)
        for (int j = lane; j < N; j += 32) {
          float g = 0.f;
          if (i < K) {
            for (int b = b0; b < b0 + nb; ++b) g = fmaf(in[(size_t)b * K + i], dout[(size_t)b * N + j], g);
            G[oW + i * N + j] = g;
          } else {
            for (int b = b0; b < b0 + nb; ++b) g += dout[(size_t)b * N + j];
            G[ob + j] = g;
          }
        }
    };
    // dh2 from the class layer
    dense_din(warp, kCnnThreads / 32, dz3, D.f2, D.ncls, w + D.oF3, h2, dh2, true);
    __syncthreads();
    // class layer gradient (warps 0-3) | dh1 through dense layer 2 (the other warps)
    if (warp < kGradW) dense_grad(warp, kGradW, h2, dz3, D.f2, D.ncls, D.oF3, D.obF3);
    else dense_din(warp - kGradW, kW - kGradW, dh2, D.f1, D.f2, w + D.oF2, h1, dh1, true);
    __syncthreads();
    // dense layer 2 gradient (first half of the warps) | dq2 through dense layer 1 (the pooled maps carry no ReLU of their own)
    if (warp < kW / 2) dense_grad(warp, kW / 2, h1, dh2, D.f1, D.f2, D.oF2, D.obF2);
    else dense_din(warp - kW / 2, kW / 2, dh1, D.flat, D.f1, w + D.oF1, q2, dq2, false);
    __syncthreads();
    // dense layer 1 gradient (all warps), then dz2 = [a2 > 0] * dq2 / 4, in place over a2
    dense_grad(warp, kW, q2, dh1, D.flat, D.f1, D.oF1, D.obF1);
    for (int e = tid; e < nb * n_a2; e += kCnnThreads) {
      const int k = b0 * n_a2 + e;
      const int x = k % D.s2, y = (k / D.s2) % D.s2, bc = k / (D.s2 * D.s2);
      const float g = dq2[((size_t)bc * D.p2 + (y >> 1)) * D.p2 + (x >> 1)];
      a2[k] = a2[k] > 0.f ? 0.25f * g : 0.f;
    }
    __syncthreads();
    // dq1[b, c1, y, x] = sum_{c2, dy, dx} dz2[b, c2, y - dy, x - dx] W2[c2, c1, dy, dx].  A work item is four
    // neighbouring outputs of a row: per (c2, dy) it reads the eight values of dz2's row y - dy that they touch
    // (off the map: a clamped address, counted as zero) and the five weights, and does twenty multiply-adds;
    // rows off the map are skipped whole.
    {
      const float* dz2 = a2;
      const float* W2 = w + D.oW2;
      const int xq = (D.p1 + 3) / 4, items = nb * D.c1 * D.p1 * xq;
      for (int e = tid; e < items; e += kCnnThreads) {
        const int x0 = (e % xq) * 4, y = (e / xq) % D.p1, c = (e / (xq * D.p1)) % D.c1, b = b0 + e / (xq * D.p1 * D.c1);
        int co[8];
        bool cok[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {   // column x0 - 4 + k of dz2
          const int xx = x0 - 4 + k;
          cok[k] = xx >= 0 && xx < D.s2;
          co[k] = min(max(xx, 0), D.s2 - 1);
        }
        float o[4] = {0.f, 0.f, 0.f, 0.f};
        for (int c2 = 0; c2 < D.c2; ++c2) {
          const float* dzp = dz2 + (size_t)(b * D.c2 + c2) * D.s2 * D.s2;
          const float* wk = W2 + (c2 * D.c1 + c) * (kK * kK);
#pragma unroll
          for (int dy = 0; dy < kK; ++dy) {
            const int yy = y - dy;
            if (yy < 0 || yy >= D.s2) continue;
            float v[8], wv[kK];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = cok[k] ? dzp[yy * D.s2 + co[k]] : 0.f;
#pragma unroll
            for (int dx = 0; dx < kK; ++dx) wv[dx] = wk[dy * kK + dx];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int dx = 0; dx < kK; ++dx) o[i] = fmaf(v[4 + i - dx], wv[dx], o[i]);   // output x0 + i takes column x0 + i - dx
          }
        }
        float* out = dq1 + ((size_t)(b * D.c1 + c) * D.p1 + y) * D.p1 + x0;
#pragma unroll
        for (int i = 0; i < 4; ++i) if (x0 + i < D.p1) out[i] = o[i];
      }
    }
    __syncthreads();
    // Second convolution's gradient.  A work item is one kernel row (c2, c, dy): its five taps share every value of
    // dz2 they meet, and the input row slides through a five-register window (two loads per five multiply-adds).
    // Then the bias gradients, and dz1 = [a1 > 0] * dq1 / 4 in place over a1.
    {
      const int nrow = D.c2 * D.c1 * kK, nd = nb * n_a1;
      const float* dz2 = a2;
      for (int e = tid; e < nrow + D.c2 + nd; e += kCnnThreads) {
        if (e < nrow) {
          const int dy = e % kK, c = (e / kK) % D.c1, c2 = e / (kK * D.c1);
          float g[kK] = {0.f, 0.f, 0.f, 0.f, 0.f};
          for (int b = b0; b < b0 + nb; ++b) {
            const float* dzp = dz2 + (size_t)(b * D.c2 + c2) * D.s2 * D.s2;
            const float* qp = q1 + ((size_t)(b * D.c1 + c) * D.p1 + dy) * D.p1;
            for (int y = 0; y < D.s2; ++y) {
              const float* qr = qp + y * D.p1;
              float q0 = qr[0], q1v = qr[1], q2v = qr[2], q3v = qr[3];
              for (int x = 0; x < D.s2; ++x) {
                const float d = dzp[y * D.s2 + x], q4v = qr[x + 4];
                g[0] = fmaf(d, q0, g[0]); g[1] = fmaf(d, q1v, g[1]); g[2] = fmaf(d, q2v, g[2]);
                g[3] = fmaf(d, q3v, g[3]); g[4] = fmaf(d, q4v, g[4]);
                q0 = q1v; q1v = q2v; q2v = q3v; q3v = q4v;
              }
            }
          }
#pragma unroll
          for (int dx = 0; dx < kK; ++dx) G[D.oW2 + e * kK + dx] = g[dx];
        } else if (e < nrow + D.c2) {
          const int c2 = e - nrow;
          float g = 0.f;
          for (int b = b0; b < b0 + nb; ++b) {
            const float* dzp = dz2 + (size_t)(b * D.c2 + c2) * D.s2 * D.s2;
            for (int k = 0; k < D.s2 * D.s2; ++k) g += dzp[k];
          }
          G[D.ob2 + c2] = g;
        } else {
          const int k = b0 * n_a1 + (e - nrow - D.c2);
          const int x = k % D.s1, y = (k / D.s1) % D.s1, bc = k / (D.s1 * D.s1);
          const float g = dq1[((size_t)bc * D.p1 + (y >> 1)) * D.p1 + (x >> 1)];
          a1[k] = a1[k] > 0.f ? 0.25f * g : 0.f;
        }
      }
    }
    __syncthreads();
    // First convolution's gradient: few parameters, long sums.  A warp takes one (output plane, input plane)
    // pair: lanes across a row of the output map, every lane all 25 taps, so that a value of dz1 (global,
    // one load per row, the rows independent of one another) meets 25 inputs from shared memory; 26
    // shuffle trees at the end (the 25 taps and, for the first input plane, the bias).
    {
      const float* dz1 = a1;
      for (int e = warp; e < D.c1 * D.cin; e += kCnnThreads / 32) {
        const int ci = e % D.cin, c = e / D.cin;
        float g[kK * kK], gb = 0.f;
#pragma unroll
        for (int k = 0; k < kK * kK; ++k) g[k] = 0.f;
        for (int b = b0; b < b0 + nb; ++b) {
          const float* dzp = dz1 + (size_t)(b * D.c1 + c) * D.s1 * D.s1;
          // input plane ci of sample b: shared memory if the rows were staged, else the client's data
          const float* xp = (rows_staged ? xs + (b - b0) * rowlen : xrows + (size_t)idx[b] * rowlen) + ci * D.side * D.side;
          for (int x = lane; x < D.s1; x += 32) {
#pragma unroll 2
            for (int y = 0; y < D.s1; ++y) {
              const float d = dzp[y * D.s1 + x];
              const float* xr = xp + y * D.side + x;
              gb += d;
#pragma unroll
              for (int dy = 0; dy < kK; ++dy)
#pragma unroll
                for (int dx = 0; dx < kK; ++dx) g[dy * kK + dx] = fmaf(d, xr[dy * D.side + dx], g[dy * kK + dx]);
            }
          }
        }
#pragma unroll
        for (int k = 0; k < kK * kK; ++k) {
#pragma unroll
          for (int m = 16; m; m >>= 1) g[k] += __shfl_xor_sync(0xffffffffu, g[k], m);
        }
#pragma unroll
        for (int m = 16; m; m >>= 1) gb += __shfl_xor_sync(0xffffffffu, gb, m);
        if (lane == 0) {
#pragma unroll
          for (int k = 0; k < kK * kK; ++k) G[D.oW1 + (c * D.cin + ci) * (kK * kK) + k] = g[k];
          if (ci == 0) G[D.ob1 + c] = gb;
        }
      }
    }
    cluster_sync();   // every CTA's partial gradients are in global scratch; nobody reads the old weights any more

    // ================= this CTA's slice: g = sum over the CTAs in rank order; w -= eta (g + lambda w), U += g + lambda w =================
    {
      const float* G0 = act + D.total;
      uint32_t peer_w[kMaxCl];   // the model's shared-memory address in every CTA of the cluster
#pragma unroll
      for (int q = 0; q < kMaxCl; ++q)
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(peer_w[q]) : "r"((uint32_t)__cvta_generic_to_shared(w)), "r"((uint32_t)(q < CL ? q : 0)));
      // four parameters per thread and trip, so that 32 loads of partials and 4 of U are in flight at once
      constexpr int kTrip = 4;
      for (int kb = k_lo + tid; kb < k_hi; kb += kTrip * kCnnThreads) {
        float part[kTrip][kMaxCl], uold[kTrip];
#pragma unroll
        for (int r = 0; r < kTrip; ++r) {
          const int k = kb + r * kCnnThreads;
#pragma unroll
          for (int q = 0; q < kMaxCl; ++q) part[r][q] = (k < k_hi && q < nact) ? G0[(size_t)q * D.Ppad + k] : 0.f;
          uold[r] = k < k_hi ? Urow[k] : 0.f;
        }
#pragma unroll
        for (int r = 0; r < kTrip; ++r) {
          const int k = kb + r * kCnnThreads;
          if (k >= k_hi) break;
          float g = 0.f;
#pragma unroll
          for (int q = 0; q < kMaxCl; ++q) g += part[r][q];
          const bool bias = (k >= D.ob1 && k < D.oW2) || (k >= D.ob2 && k < D.oF1) || (k >= D.obF1 && k < D.oF2) ||
                            (k >= D.obF2 && k < D.oF3) || k >= D.obF3;   // biases take no l2 term
          const float wk = w[k];
          const float gt = bias ? g : fmaf(lambda, wk, g);
          const float wn = fmaf(-eta, gt, wk);
          Urow[k] = uold[r] + gt;
#pragma unroll
          for (int q = 0; q < kMaxCl; ++q)
            if (q < CL) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(peer_w[q] + 4u * (uint32_t)k), "f"(wn) : "memory");
        }
      }
    }
    cluster_sync();   // the new weights are in every CTA's copy
  }

  // ---- event trigger: h reached s_{i,c}; U_i is complete in its row; the end model on request ----
  if (p.r.w_end) {
    float* dst = p.r.w_end + (size_t)t.u_row * p.r.stride;
    for (int k = k_lo + tid; k < k_hi; k += kCnnThreads) dst[k] = w[k];
  }
  if (tid == 0 && rank == 0) {
    TriggerRec rec;
    rec.client = t.client; rec.round = t.round; rec.samples_done = t.steps * (uint32_t)B; rec.flags = 1;
    p.r.trig[t.seq] = rec;
  }
}

size_t cnn_smem_bytes(const CnnShape& s) {
  const CnnDims d = make_cnn_dims(s);
  return ((size_t)((d.P + 3) & ~3) + 2 * s.batch) * sizeof(float);
}
// with room for the minibatch rows of one CTA of a cluster of `cl` and, if `acts`, for its small activations
// (0 if they do not fit)
size_t cnn_smem_bytes_staged(const CnnShape& s, uint32_t cl, bool acts) {
  const CnnDims d = make_cnn_dims(s);
  const size_t per = (s.batch + cl - 1) / cl;
  const size_t extra = per * ((size_t)d.cin * d.side * d.side + (acts ? (size_t)cnn_small_acts(d) : 0)) * sizeof(float);
  const size_t all = cnn_smem_bytes(s) + extra;
  return all <= 227 * 1024 ? all : 0;
}

}  // namespace

uint32_t cnn_n_params(const CnnShape& s) { return (uint32_t)make_cnn_dims(s).P; }
// activations of a minibatch, then one row of gradient partials per CTA of the cluster
size_t cnn_act_floats(const CnnShape& s) {
  const CnnDims d = make_cnn_dims(s);
  return (size_t)d.total + (size_t)kMaxCl * d.Ppad;
}

const char* cnn_check_shape(const CnnShape& s) {
  const int side = (int)s.dims[0];
  const int s1 = side - kK + 1;
  if (side < 2 * kK || s1 <= 0 || (s1 & 1)) return "convolutional model: (side - 4) must be even and positive";
  const int s2 = s1 / 2 - kK + 1;
  if (s2 <= 0 || (s2 & 1)) return "convolutional model: ((side - 4) / 2 - 4) must be even and positive";
  for (int i = 1; i < 7; ++i) if (s.dims[i] == 0) return "convolutional model: a width is zero";
  if (s.dims[6] > 32) return "at most 32 classes are supported";
  if (s.batch == 0 || s.batch > 64) return "convolutional model: batch must be 1 .. 64";
  if (cnn_smem_bytes(s) > 220 * 1024) return "convolutional model: the parameters do not fit in shared memory (about 55,000)";
  return nullptr;
}

cudaError_t launch_cnn_rounds(const CnnLaunch& p0, cudaStream_t s) {
  if (p0.r.n_tasks == 0) return cudaSuccess;
  int sms = 0;   // asked of the current device at every launch: cheap, and right on any device of the process
  {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  // CTAs per round-task: as many as the minibatch has samples and the launch leaves SMs for
  uint32_t cl = kMaxCl;
  while (cl > 1 && (cl > p0.shape.batch || p0.r.n_tasks * cl > (uint32_t)sms)) cl >>= 1;
  CnnLaunch p = p0;
  size_t smem = cnn_smem_bytes_staged(p.shape, cl, true);
  p.stage_acts = smem != 0;
  if (!smem) smem = cnn_smem_bytes_staged(p.shape, cl, false);
  p.stage_rows = smem != 0;
  if (!smem) smem = cnn_smem_bytes(p.shape);
  bool fixed = cl == kMaxCl && p.stage_acts && p.shape.batch == kLeNetShape.batch;
  for (int i = 0; i < 7; ++i) fixed = fixed && p.shape.dims[i] == kLeNetShape.dims[i];
  cudaError_t e = cudaFuncSetAttribute(fixed ? cnn_round_kernel<true> : cnn_round_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.r.n_tasks * cl, 1, 1);
  cfg.blockDim = dim3(kCnnThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return fixed ? cudaLaunchKernelEx(&cfg, cnn_round_kernel<true>, p) : cudaLaunchKernelEx(&cfg, cnn_round_kernel<false>, p);
}

}  // namespace aet
