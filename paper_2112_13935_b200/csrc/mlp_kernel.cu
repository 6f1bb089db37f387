// Local-SGD round of one client for a ReLU MLP with minibatches.
//
// Algorithm 3, MainComputeNode, inner loop with xi a minibatch of B samples:
// g = mean gradient; w_c -= eta_i * g; U_i += g.  One thread-block cluster runs
// one round-task.  Every layer's weight matrix W_l [in, out] is split by input
// rows over the cluster's CTAs: CTA r owns rows_r(l), and is the only one that
// ever reads or writes them (master copy and update sum stay in its part of
// global memory / L2).  Per SGD iteration:
//   forward  l = 0..L-1: partial_l[r] = A_{l-1}[:, rows_r] * W_l[rows_r, :]
//            -> cluster barrier -> each CTA sums the partials of the columns it
//            needs next, adds the bias, applies ReLU (last layer: softmax and
//            dZ = (p - onehot) / B, computed by every CTA);
//   backward l = L-1..0: dZ_{l-1}[:, rows_r] = (dZ_l * W_l[rows_r, :]^T) * relu'
//            and, fused on the same staged tiles, g = A_{l-1}[:, rows_r]^T dZ_l
//            (+ lambda W), W -= eta g, U += g -> cluster barrier.
// precision 1 rounds to bf16 where a bf16 tensor-core path would: the inputs
// (at load), W_l on every read, hidden activations after ReLU, dZ_l before the
// two backward products; sums, bias gradients and the master update are fp32.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"
#include "mlp_common.cuh"

namespace aet {
namespace {

using namespace mlp;

constexpr int kThreads = 512;
constexpr int kRC = 32;        // rows of W_l staged per chunk
constexpr int kMaxTiles = 2;   // 4x4 output micro-tiles per thread in the forward product

struct Smem {  // offsets (in floats) into dynamic shared memory
  int idx, As, AsT, Ws, dzs, dzq, zs, total;
};
__host__ __device__ inline Smem make_smem(const MlpShape& s) {
  int Bp = (s.batch + 3) & ~3, nmax = 0;
  for (uint32_t l = 0; l < s.n_layers; ++l) nmax = max(nmax, (int)((s.dims[l + 1] + 3) & ~3u));
  Smem m{};
  int o = 0;
  m.idx = o; o += Bp;
  m.As = o; o += kRC * Bp;
  m.AsT = o; o += Bp * kRC;
  m.Ws = o; o += kRC * (nmax + 4);
  m.dzs = o; o += Bp * nmax;
  m.dzq = o; o += (s.precision == 1) ? Bp * nmax : 0;
  m.zs = o; o += Bp * 32;
  m.total = o;
  return m;
}

template <class Load, class Store>
__device__ __forceinline__ void staged_copy(int total, int tid, Load ld, Store st) {
  staged_copy_t<kThreads>(total, tid, ld, st);
}

__global__ void __launch_bounds__(kThreads) mlp_round_kernel(MlpLaunch p) {
  extern __shared__ __align__(16) float sm[];
  const MlpShape& S = p.shape;
  const int C = (int)S.cluster;
  const bool clustered = C > 1;
  const int rank = clustered ? (int)cluster_rank() : 0;
  const TaskDesc t = p.r.tasks[p.r.task_begin + blockIdx.x / C];
  if (!debug_task_ok(p.r, t)) return;   // debug checks only: rows and slots in range, else flag and skip
  if (t.n_samples == 0) {   // an empty round (every CTA of the cluster takes this branch)
    if (rank == 0) {
      uint32_t P = 0;
      for (uint32_t l = 0; l < S.n_layers; ++l) P += S.dims[l] * S.dims[l + 1] + S.dims[l + 1];
      publish_empty_round(p.r, t, P);
    }
    return;
  }
  const int tid = threadIdx.x;
  const int L = (int)S.n_layers, B = (int)S.batch, Bp = up4(B);
  const bool bf = S.precision == 1;
  const Smem M = make_smem(S);
  const Layout G = make_layout(S);
  int* idx = reinterpret_cast<int*>(sm + M.idx);
  float* As = sm + M.As;
  float* AsT = sm + M.AsT;
  float* Ws = sm + M.Ws;
  float* dzs = sm + M.dzs;
  float* dzq = bf ? sm + M.dzq : dzs;
  float* zs = sm + M.zs;

  float* act = p.act + (size_t)(blockIdx.x / C) * p.act_stride;
  float* work = p.work + (size_t)t.client * p.r.stride;
  float* Urow = p.r.U + (size_t)t.u_row * p.r.stride;
  const ClientData cd = p.r.clients[t.client];
  const uint64_t key = p.r.sample_keys[t.client];
  const float eta = t.eta, lambda = p.r.l2;

  // parameter offsets and this CTA's row slice of every layer
  size_t woff[AET_MAX_LAYERS], boff[AET_MAX_LAYERS];
  int r0[AET_MAX_LAYERS], r1[AET_MAX_LAYERS];
  {
    size_t o = 0;
    for (int l = 0; l < L; ++l) {
      woff[l] = o; o += (size_t)S.dims[l] * S.dims[l + 1];
      boff[l] = o; o += S.dims[l + 1];
      r0[l] = (int)(((long long)S.dims[l] * rank) / C);
      r1[l] = (int)(((long long)S.dims[l] * (rank + 1)) / C);
    }
  }

  // ---- start model into the client's work row: snapshot - own in-flight sums ----
  {
    const float* snap = p.r.snaps + (size_t)t.snap_slot * p.r.stride;
    for (int l = 0; l < L; ++l) {
      const int N = (int)S.dims[l + 1];
      const size_t lo = woff[l] + (size_t)r0[l] * N, hi = woff[l] + (size_t)r1[l] * N;
      for (size_t j = lo + tid; j < hi; j += kThreads) {
        float w = snap[j];
        for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
          const InflightRef ref = p.r.inflight[t.inflight_off + f];
          w = fmaf(-ref.eta, p.r.U[(size_t)ref.row * p.r.stride + j], w);
        }
        work[j] = w;
        Urow[j] = 0.f;
      }
      if (rank == l % C)
        for (int j = tid; j < N; j += kThreads) {
          float w = snap[boff[l] + j];
          for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
            const InflightRef ref = p.r.inflight[t.inflight_off + f];
            w = fmaf(-ref.eta, p.r.U[(size_t)ref.row * p.r.stride + boff[l] + j], w);
          }
          work[boff[l] + j] = w;
          Urow[boff[l] + j] = 0.f;
        }
    }
  }
  cluster_sync(clustered);

  uint32_t h = 0;  // local sample counter of Algorithm 3
  for (uint32_t it = 0; it < t.steps; ++it) {
    for (int b = tid; b < Bp; b += kThreads)
      idx[b] = b < B ? (int)sample_index(draw(key, t.sample_ctr0 + (uint64_t)it * B + b), cd.n) : 0;
    __syncthreads();

    // ================= forward =================
    for (int l = 0; l < L; ++l) {
      const int N = (int)S.dims[l + 1], Np = up4(N), ldw = Np + 4;
      const int tiles_n = Np / 4, tiles = (Bp / 4) * tiles_n;
      float acc[kMaxTiles][16];
#pragma unroll
      for (int q = 0; q < kMaxTiles; ++q)
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[q][e] = 0.f;

      for (int c0 = r0[l]; c0 < r1[l]; c0 += kRC) {
        const int rc = min(kRC, r1[l] - c0);
        __syncthreads();
        // stage A chunk as As[ic][b] and W chunk as Ws[ic][j]
        staged_copy(kRC * Bp, tid,
                    [&](int e) {
                      const int b = e / kRC, ic = e % kRC;
                      if (b >= B || ic >= rc) return 0.f;
                      if (l > 0) return act[G.a[l - 1] + (size_t)b * S.dims[l] + c0 + ic];
                      const size_t off = (size_t)idx[b] * S.dims[0] + c0 + ic;
                      return bf ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(cd.x)[off])
                                : reinterpret_cast<const float*>(cd.x)[off];
                    },
                    [&](int e, float v) { As[(e % kRC) * Bp + e / kRC] = v; });
        staged_copy(kRC * Np, tid,
                    [&](int e) {
                      const int ic = e / Np, j = e % Np;
                      if (ic >= rc || j >= N) return 0.f;
                      const float v = work[woff[l] + (size_t)(c0 + ic) * N + j];
                      return bf ? q_bf16(v) : v;
                    },
                    [&](int e, float v) { Ws[(e / Np) * ldw + e % Np] = v; });
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxTiles; ++q) {
          const int mt = tid + q * kThreads;
          if (mt < tiles) {
            const int bt = mt / tiles_n, jt = mt % tiles_n;
            for (int ic = 0; ic < rc; ++ic) {
              const float4 a = *reinterpret_cast<const float4*>(As + ic * Bp + 4 * bt);
              const float4 w = *reinterpret_cast<const float4*>(Ws + ic * ldw + 4 * jt);
              const float av[4] = {a.x, a.y, a.z, a.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[q][4 * i + j] = fmaf(av[i], wv[j], acc[q][4 * i + j]);
            }
          }
        }
      }
      // partial sums of this CTA -> global scratch
      {
        float* part = act + G.part[l] + (size_t)rank * B * N;
#pragma unroll
        for (int q = 0; q < kMaxTiles; ++q) {
          const int mt = tid + q * kThreads;
          if (mt < tiles) {
            const int bt = mt / tiles_n, jt = mt % tiles_n;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int b = 4 * bt + i, n = 4 * jt + j;
                if (b < B && n < N) part[(size_t)b * N + n] = acc[q][4 * i + j];
              }
          }
        }
      }
      cluster_sync(clustered);
      const float* part0 = act + G.part[l];
      const float* bias = work + boff[l];
      if (l < L - 1) {
        // columns this CTA feeds into the next layer
        const int c_lo = r0[l + 1], c_n = r1[l + 1] - r0[l + 1];
        staged_copy(B * c_n, tid,
                    [&](int e) {
                      const int b = e / c_n, n = c_lo + e % c_n;
                      float z = bias[n];
                      for (int r = 0; r < C; ++r) z += part0[((size_t)r * B + b) * N + n];
                      return z;
                    },
                    [&](int e, float z) {
                      const float a = fmaxf(z, 0.f);
                      act[G.a[l] + (size_t)(e / c_n) * N + c_lo + e % c_n] = bf ? q_bf16(a) : a;
                    });
        __syncthreads();
      } else {
        staged_copy(B * N, tid,
                    [&](int e) {
                      const int b = e / N, n = e % N;
                      float z = bias[n];
                      for (int r = 0; r < C; ++r) z += part0[((size_t)r * B + b) * N + n];
                      return z;
                    },
                    [&](int e, float z) { zs[(e / N) * 32 + e % N] = z; });
        __syncthreads();
        // softmax cross-entropy: dZ = (p - onehot(y)) / B
        for (int b = tid; b < Bp; b += kThreads) {
          if (b < B) {
            float m = -INFINITY;
            for (int n = 0; n < N; ++n) m = fmaxf(m, zs[b * 32 + n]);
            float sum = 0.f;
            for (int n = 0; n < N; ++n) sum += __expf(zs[b * 32 + n] - m);
            const int y = cd.y[idx[b]];
            const float inv = 1.f / sum, invB = 1.f / (float)B;
            for (int n = 0; n < Np; ++n) {
              float d = 0.f;
              if (n < N) d = (__expf(zs[b * 32 + n] - m) * inv - (n == y ? 1.f : 0.f)) * invB;
              dzs[b * Np + n] = d;
              if (bf) dzq[b * Np + n] = q_bf16(d);
            }
          } else {
            for (int n = 0; n < Np; ++n) { dzs[b * Np + n] = 0.f; if (bf) dzq[b * Np + n] = 0.f; }
          }
        }
        __syncthreads();
      }
    }

    // ================= backward + update =================
    for (int l = L - 1; l >= 0; --l) {
      const int N = (int)S.dims[l + 1], Np = up4(N), ldw = Np + 4;
      const int K = (int)S.dims[l];
      for (int c0 = r0[l]; c0 < r1[l]; c0 += kRC) {
        const int rc = min(kRC, r1[l] - c0);
        __syncthreads();
        staged_copy(kRC * Bp, tid,
                    [&](int e) {
                      const int b = e / kRC, ic = e % kRC;
                      if (b >= B || ic >= rc) return 0.f;
                      if (l > 0) return act[G.a[l - 1] + (size_t)b * K + c0 + ic];
                      const size_t off = (size_t)idx[b] * S.dims[0] + c0 + ic;
                      return bf ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(cd.x)[off])
                                : reinterpret_cast<const float*>(cd.x)[off];
                    },
                    [&](int e, float v) { AsT[e] = v; });
        if (l > 0)
          staged_copy(kRC * Np, tid,
                      [&](int e) {
                        const int ic = e / Np, j = e % Np;
                        if (ic >= rc || j >= N) return 0.f;
                        const float v = work[woff[l] + (size_t)(c0 + ic) * N + j];
                        return bf ? q_bf16(v) : v;
                      },
                      [&](int e, float v) { Ws[(e / Np) * ldw + e % Np] = v; });
        __syncthreads();
        if (l > 0) {
          // dZ_{l-1}[b, c0+ic] = relu'(A_{l-1}) * sum_j dZq_l[b, j] W_l[c0+ic, j]
          for (int e = tid; e < B * rc; e += kThreads) {
            const int b = e / rc, ic = e % rc;
            float s = 0.f;
            for (int j = 0; j < Np; j += 4) {
              const float4 d = *reinterpret_cast<const float4*>(dzq + b * Np + j);
              const float4 w = *reinterpret_cast<const float4*>(Ws + ic * ldw + j);
              s = fmaf(d.x, w.x, s); s = fmaf(d.y, w.y, s); s = fmaf(d.z, w.z, s); s = fmaf(d.w, w.w, s);
            }
            const float a = AsT[b * kRC + ic];
            act[G.dz[l - 1] + (size_t)b * K + c0 + ic] = a > 0.f ? s : 0.f;
          }
        }
        // g[c0+ic, j] = sum_b A[b, c0+ic] dZq_l[b, j] (+ lambda W); W -= eta g; U += g
        {
          const int tiles_n = Np / 4, tiles = (kRC / 4) * tiles_n;
          for (int mt = tid; mt < tiles; mt += kThreads) {
            const int it4 = mt / tiles_n, jt = mt % tiles_n;
            float g[16], wv[16], uv[16];
#pragma unroll
            for (int i = 0; i < 4; ++i)     // master and update-sum entries first: in flight during the FMAs
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int ic = 4 * it4 + i, n = 4 * jt + j;
                const bool live = ic < rc && n < N;
                const size_t o = woff[l] + (size_t)(c0 + ic) * N + n;
                wv[4 * i + j] = live ? work[o] : 0.f;
                uv[4 * i + j] = live ? Urow[o] : 0.f;
              }
#pragma unroll
            for (int e = 0; e < 16; ++e) g[e] = 0.f;
            for (int b = 0; b < B; ++b) {
              const float4 a = *reinterpret_cast<const float4*>(AsT + b * kRC + 4 * it4);
              const float4 d = *reinterpret_cast<const float4*>(dzq + b * Np + 4 * jt);
              const float av[4] = {a.x, a.y, a.z, a.w}, dv[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
              for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) g[4 * i + j] = fmaf(av[i], dv[j], g[4 * i + j]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int ic = 4 * it4 + i;
              if (ic >= rc) continue;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int n = 4 * jt + j;
                if (n >= N) continue;
                const size_t o = woff[l] + (size_t)(c0 + ic) * N + n;
                const float w = wv[4 * i + j];
                const float gg = fmaf(lambda, w, g[4 * i + j]);
                work[o] = fmaf(-eta, gg, w);
                Urow[o] = uv[4 * i + j] + gg;
              }
            }
          }
        }
      }
      cluster_sync(clustered);
      // bias of layer l: its owner updates it once everybody has read it
      if (rank == l % C)
        for (int n = tid; n < N; n += kThreads) {
          float gb = 0.f;
          for (int b = 0; b < B; ++b) gb += dzs[b * Np + n];
          work[boff[l] + n] = fmaf(-eta, gb, work[boff[l] + n]);
          Urow[boff[l] + n] += gb;
        }
      if (l > 0) {
        __syncthreads();
        const int Nm = (int)S.dims[l], Nmp = up4(Nm);
        staged_copy(Bp * Nmp, tid,
                    [&](int e) {
                      const int b = e / Nmp, n = e % Nmp;
                      return (b < B && n < Nm) ? act[G.dz[l - 1] + (size_t)b * Nm + n] : 0.f;
                    },
                    [&](int e, float d) { dzs[e] = d; if (bf) dzq[e] = q_bf16(d); });
        __syncthreads();
      }
    }
    h += (uint32_t)B;
  }

  // ---- event trigger: publish (c, U_i, i) ----
  cluster_sync(clustered);
  if (p.r.w_end) {
    float* dst = p.r.w_end + (size_t)t.u_row * p.r.stride;
    for (int l = 0; l < L; ++l) {
      const int N = (int)S.dims[l + 1];
      const size_t lo = woff[l] + (size_t)r0[l] * N, hi = woff[l] + (size_t)r1[l] * N;
      for (size_t j = lo + tid; j < hi; j += kThreads) dst[j] = work[j];
      if (rank == l % C)
        for (int j = tid; j < N; j += kThreads) dst[boff[l] + j] = work[boff[l] + j];
    }
  }
  if (rank == 0 && tid == 0) {
    TriggerRec rec;
    rec.client = t.client; rec.round = t.round; rec.samples_done = h; rec.flags = 1;
    p.r.trig[t.seq] = rec;
  }
}

}  // namespace

size_t mlp_act_floats(const MlpShape& shape) { return make_layout(shape).total; }

const char* mlp_check_shape(const MlpShape& shape) {
  const int Bp = (shape.batch + 3) & ~3u;
  for (uint32_t l = 0; l < shape.n_layers; ++l) {
    const int Np = (shape.dims[l + 1] + 3) & ~3u;
    if ((Bp / 4) * (Np / 4) > kMaxTiles * kThreads) return "batch * layer width exceeds 16384";
  }
  if ((size_t)make_smem(shape).total * sizeof(float) > 227 * 1024) return "layer widths need more shared memory than a CTA has";
  return nullptr;
}

uint32_t mlp_pick_cluster(const MlpShape& shape, uint32_t n_clients) {
  uint32_t c = 8;
  while (c > 1 && (uint64_t)n_clients * c > 148) c >>= 1;
  (void)shape;
  return c;
}

cudaError_t launch_mlp_rounds(const MlpLaunch& p, cudaStream_t s) {
  if (p.r.n_tasks == 0) return cudaSuccess;
  if (mlp_stream_eligible(p.shape)) return launch_mlp_stream_rounds(p, s);
  if (mlp_tc_eligible(p.shape)) return launch_mlp_tc_rounds(p, s);
  if (mlp_res_eligible(p)) return launch_mlp_res_rounds(p, s);
  const Smem m = make_smem(p.shape);
  const size_t smem = (size_t)m.total * sizeof(float);
  // The shared-memory opt-in is a per-device attribute of the kernel and cheap to set: set it on
  // every launch rather than caching it per process (a second device, or two host threads).
  {
    cudaError_t e = cudaFuncSetAttribute(mlp_round_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.r.n_tasks * p.shape.cluster, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.shape.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, mlp_round_kernel, p);
}

}  // namespace aet
