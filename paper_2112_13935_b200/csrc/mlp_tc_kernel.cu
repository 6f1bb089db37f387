// Local-SGD round of one client for a bf16-operand ReLU MLP: the two products
// of the wide first layer run on the 5th-generation tensor cores.
//
// Algorithm 3, MainComputeNode, inner loop with xi a minibatch (mean gradient;
// w_c -= eta_i g; U_i += g).  Same cluster structure as the fp32 kernel: every
// W_l is split by input rows over the CTAs of the round-task's cluster.  What
// changes is layer 0, which carries ~95 % of the flops of a 3072-256-128-10 net:
//   forward   Z0^T[out0 x B] += W0[rows]^T . X[:, rows]^T: A = bf16(W0 chunk)^T, B = X chunk
//             [B x rows]; tcgen05.mma M = 128 (x out0/128), N = B, fp32 accumulators in TMEM.
//             Only the first iteration of a round runs it as a pass of its own (chunks of 64
//             rows converted from the fp32 master, tiles double-buffered, completion by
//             tcgen05.commit on mbarriers); afterwards the product for iteration t + 1 is
//             issued from inside the backward pass of iteration t, chunk by chunk, from the
//             weights that pass has just updated, so W0 is read once per iteration, not twice;
//   backward  G[128 rows x out0] = X[:, rows]^T . dZ0       chunks of 128 input rows, in units
//             of 128 columns: A = X chunk^T [128 x B], B = bf16(dZ0)^T [128 x B]; M = 128,
//             N = 128, K = B; two TMEM slots so the MMAs of unit u+1 run while the epilogue
//             of unit u reads its tile back (tcgen05.ld) and does g = G + lambda W,
//             W -= eta g on the fp32 master in HBM/L2.
// Operand tiles use the K-major, no-swizzle core-matrix layout (8 rows x 16 bytes
// contiguous; LBO = stride between core matrices along K, SBO = along M/N).
// The narrow layers (l >= 1), softmax and bias updates run on plain FMAs.
// Every mbarrier wait is bounded; after a timeout the CTA flags `status`, stops
// polling and keeps to the barrier schedule so that its cluster peers never block.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"
#include "mlp_common.cuh"

namespace aet {
namespace {

using namespace mlp;

constexpr int kThreads = 512;   // 16 warps: enough loads in flight to cover HBM/L2 latency
constexpr int kColSplit = kThreads / 128;  // warps sharing one 32-lane quarter of tensor memory split the columns
constexpr int kRC = 32;        // rows per chunk of the FMA layers
constexpr int kMaxTiles = 2;
constexpr int kKC = 64;        // input rows per forward chunk
constexpr int kMT = 128;       // input rows per backward chunk (M of the MMA)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kFwdCol = 256;   // tensor-memory columns [256, 384): layer-0 forward accumulators
constexpr int kTrLd = 36;     // floats per row of the epilogue transpose buffer (16-byte aligned, conflict-free)
constexpr uint32_t kWaitLimit = 1u << 22;
// The widest layer's update sum is not accumulated entry by entry: Algorithm 3 does
// w -= eta * g and U += g in the same step with eta constant within the round, so
// U_i = (w_start - w_end) / eta_i holds term by term.  The row of U keeps w_start during
// the round and is turned into U_i at the event trigger; this removes the read and the
// write of U_0 (40 % of the HBM traffic) from every SGD iteration.  In fp32 the quotient
// carries the rounding of the master updates (about 1e-4 of max|U| here), which is inside
// the noise of the bf16 operand roundings of this path; the fp32 kernels accumulate U.
constexpr bool kDeriveU0 = true;

struct TcSmem {  // byte offsets into dynamic shared memory
  int tiles, idx, As, AsT, Ws, dzs, dzq, zs, tr, x2, total;
};
// Operand-tile region: the larger of the stand-alone forward pass (two A and two B tiles of 64
// input rows) and the layer-0 backward pass (two X^T tiles, bf16(dZ0)^T, and for the forward
// product of the next iteration one tile of updated weights and one tile of next-batch inputs).
__host__ __device__ inline int tc_tiles_bytes(const MlpShape& s) {
  const int B = (int)s.batch, out0 = (int)s.dims[1];
  const int fwd = 2 * out0 * kKC * 2 + 2 * B * kKC * 2;
  const int bwd = 2 * kMT * B * 2 + out0 * B * 2 + 128 * kMT * 2 + B * kMT * 2;
  return max(fwd, bwd);
}
__host__ __device__ inline TcSmem make_tc_smem(const MlpShape& s) {
  const int B = (int)s.batch;
  int nmax = 0;
  for (uint32_t l = 1; l < s.n_layers; ++l) nmax = max(nmax, (int)((s.dims[l + 1] + 3) & ~3u));
  TcSmem m{};
  int o = 0;
  m.tiles = o; o += tc_tiles_bytes(s);
  m.idx = o; o += 2 * B * 4;   // sample indices of this iteration and of the next
  m.As = o; o += kRC * B * 4;
  m.AsT = o; o += B * kRC * 4;
  m.Ws = o; o += kRC * (nmax + 4) * 4;
  m.dzs = o; o += B * nmax * 4;
  m.dzq = o; o += B * nmax * 4;
  m.zs = o; o += B * 32 * 4;
  // the transposes reuse the FMA layers' staging area (idle during the layer-0 backward pass)
  // and are followed by the second tile of next-batch inputs
  m.tr = m.As;
  m.x2 = m.As + (kThreads / 32) * 32 * kTrLd * 4;
  if (o < m.x2 + B * kMT * 2) o = m.x2 + B * kMT * 2;
  m.total = o;
  return m;
}

// Can layer l of this shape use the tensor-core path?  (Rows are split evenly over the cluster.)
__host__ __device__ inline bool tc_layer_ok(const MlpShape& s, int l) {
  const int out = (int)s.dims[l + 1], rows = (int)(s.dims[l] / s.cluster), B = (int)s.batch;
  if (l == 0) return true;                       // checked by mlp_tc_eligible
  if (l == (int)s.n_layers - 1) return false;    // the class layer is too narrow for a 128-row tile
  if (out != 128 && out != 256) return false;
  if (s.dims[l] % s.cluster || rows % 128) return false;
  const int region = tc_tiles_bytes(s);
  return (128 + B) * out * 2 <= region && 2 * out * kKC * 2 + 2 * B * kKC * 2 <= region &&
         2 * kMT * B * 2 + out * B * 2 <= region;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor: K-major, no swizzle.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major.
__device__ __forceinline__ uint32_t umma_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <class Load, class Store>
__device__ __forceinline__ void staged_copy(int total, int tid, Load ld, Store st) {
  staged_copy_t<kThreads>(total, tid, ld, st);
}

// One mbarrier that tcgen05.commit arrives on, with the bookkeeping that keeps
// waits and completions paired (never more than one completion ahead).
struct CommitBar {
  uint64_t* bar;
  uint32_t issued, waited;
};
__device__ __forceinline__ void bar_drain(CommitBar& b, bool& failed) {
  while (b.waited < b.issued) {
    const uint32_t parity = b.waited & 1u;
    bool ok = failed;  // after a timeout: stop polling, keep the counters moving
    for (uint32_t i = 0; i < kWaitLimit && !ok; ++i) {
      uint32_t p;
      asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                   : "=r"(p) : "r"(smem_u32(b.bar)), "r"(parity) : "memory");
      ok = p != 0;
    }
    if (!ok) failed = true;
    ++b.waited;
  }
}

__global__ void __launch_bounds__(kThreads, 1) mlp_tc_kernel(MlpLaunch p) {
  extern __shared__ __align__(1024) unsigned char smraw[];
  __shared__ __align__(8) uint64_t bars[5];
  __shared__ uint32_t tmem_base_s;

  const MlpShape& S = p.shape;
  const int C = (int)S.cluster;
  const bool clustered = C > 1;
  const int rank = clustered ? (int)cluster_rank() : 0;
  const TaskDesc t = p.r.tasks[p.r.task_begin + blockIdx.x / C];
  if (!debug_task_ok(p.r, t)) return;   // debug checks only: rows and slots in range, else flag and skip
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int L = (int)S.n_layers, B = (int)S.batch;
  const int D0 = (int)S.dims[0];
  const TcSmem M = make_tc_smem(S);
  const Layout G = make_layout(S);
  unsigned char* tiles = smraw + M.tiles;
  int* idxbuf = reinterpret_cast<int*>(smraw + M.idx);
  float* As = reinterpret_cast<float*>(smraw + M.As);
  float* AsT = reinterpret_cast<float*>(smraw + M.AsT);
  float* Ws = reinterpret_cast<float*>(smraw + M.Ws);
  float* dzs = reinterpret_cast<float*>(smraw + M.dzs);
  float* dzq = reinterpret_cast<float*>(smraw + M.dzq);
  float* zs = reinterpret_cast<float*>(smraw + M.zs);
  float* trbuf = reinterpret_cast<float*>(smraw + M.tr);   // per-warp transpose buffers of the layer-0 epilogue

  float* act = p.act + (size_t)(blockIdx.x / C) * p.act_stride;
  float* work = p.work + (size_t)t.client * p.r.stride;
  float* Urow = p.r.U + (size_t)t.u_row * p.r.stride;
  const ClientData cd = p.r.clients[t.client];
  const __nv_bfloat16* xdata = reinterpret_cast<const __nv_bfloat16*>(cd.x);
  const uint64_t key = p.r.sample_keys[t.client];
  const float eta = t.eta, lambda = p.r.l2;

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

  // ---- barriers and tensor memory ----
  if (tid == 0) {
    for (int i = 0; i < 5; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[i])));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_base_s;
  CommitBar fbar[2] = {{&bars[0], 0, 0}, {&bars[1], 0, 0}};
  CommitBar bbar[2] = {{&bars[2], 0, 0}, {&bars[3], 0, 0}};
  CommitBar fwbar = {&bars[4], 0, 0};   // forward MMAs issued from inside the layer-0 backward pass
  bool failed = false;

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
        Urow[j] = (kDeriveU0 && l == 0) ? w : 0.f;
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

  // Layers whose products run on tensor cores: layer 0 always; a hidden layer when its width
  // and this CTA's slice of its rows fit the 128-row tiles and the operand tile region.
  bool tc_layer[AET_MAX_LAYERS];
  for (int l = 0; l < L; ++l) tc_layer[l] = tc_layer_ok(S, l);
  const uint32_t sbo_k64 = (kKC / 8) * 128;   // tiles with K = 64: next 8-row group after 8 core matrices
  const uint32_t sbo_kB = (B / 8) * 128;      // tiles with K = B
  uint32_t h = 0;

  for (uint32_t it = 0; it < t.steps; ++it) {
    // The forward product of layer 0 for iteration it + 1 is folded into the backward pass of
    // iteration it (see bwd0), so the next batch's sample indices are drawn one iteration early.
    int* idx = idxbuf + (it & 1) * B;
    int* idxn = idxbuf + ((it + 1) & 1) * B;
    const bool fuse = it + 1 < t.steps;
    for (int b = tid; b < B; b += kThreads) {
      if (it == 0) idx[b] = (int)sample_index(draw(key, t.sample_ctr0 + b), cd.n);
      if (fuse) idxn[b] = (int)sample_index(draw(key, t.sample_ctr0 + (uint64_t)(it + 1) * B + b), cd.n);
    }
    __syncthreads();

    // ================= forward of one layer on tensor cores =================
    // acc_ready: the accumulators were already filled (layer 0, by the previous backward pass)
    auto fwd_tc = [&](const int l, const bool acc_ready) {
      const int out0 = (int)S.dims[l + 1], Kin = (int)S.dims[l], R0 = r1[l] - r0[l];
      const int n_mt = out0 / 128;
      const uint32_t idesc = umma_idesc(128, B);
      const int a_bytes = out0 * kKC * 2, b_bytes = B * kKC * 2;
      const uint32_t dcol = l == 0 ? kFwdCol : 0u;
      for (int c = 0; !acc_ready && c * kKC < R0; ++c) {
        const int s = c & 1, c0 = r0[l] + c * kKC;
        unsigned char* tA = tiles + s * a_bytes;
        unsigned char* tB = tiles + 2 * a_bytes + s * b_bytes;
        bar_drain(fbar[s], failed);  // the MMAs that last read this buffer are done
        // A: bf16(W0[c0 + k, j]) as element (row j, col k)
        for (int e0 = tid; e0 < out0 * (kKC / 8); e0 += 2 * kThreads) {
          float f[2][8];
#pragma unroll
          for (int u4 = 0; u4 < 2; ++u4) {   // out0 * 8 is a multiple of 2 * kThreads: no tail
            const int e = e0 + u4 * kThreads, j = e % out0, kg = e / out0;
            const float* src = work + woff[l] + (size_t)(c0 + kg * 8) * out0 + j;
#pragma unroll
            for (int k = 0; k < 8; ++k) f[u4][k] = src[(size_t)k * out0];
          }
#pragma unroll
          for (int u4 = 0; u4 < 2; ++u4) {
            const int e = e0 + u4 * kThreads, j = e % out0, kg = e / out0;
            uint4 v;
            v.x = pack_bf16(f[u4][0], f[u4][1]); v.y = pack_bf16(f[u4][2], f[u4][3]);
            v.z = pack_bf16(f[u4][4], f[u4][5]); v.w = pack_bf16(f[u4][6], f[u4][7]);
            *reinterpret_cast<uint4*>(tA + (j >> 3) * sbo_k64 + kg * 128 + (j & 7) * 16) = v;
          }
        }
        // B: the layer's input, element (row b, col k): X[idx[b], c0 + k] (bf16 in HBM) or A_{l-1}[b, c0 + k]
        for (int e = tid; e < B * (kKC / 8); e += kThreads) {
          const int kg = e % (kKC / 8), b = e / (kKC / 8);
          uint4 v;
          if (l == 0) {
            v = __ldg(reinterpret_cast<const uint4*>(xdata + (size_t)idx[b] * D0 + c0 + kg * 8));
          } else {
            const float4* src = reinterpret_cast<const float4*>(act + G.a[l - 1] + (size_t)b * Kin + c0 + kg * 8);
            const float4 lo = src[0], hi = src[1];
            v.x = pack_bf16(lo.x, lo.y); v.y = pack_bf16(lo.z, lo.w); v.z = pack_bf16(hi.x, hi.y); v.w = pack_bf16(hi.z, hi.w);
          }
          *reinterpret_cast<uint4*>(tB + (b >> 3) * sbo_k64 + kg * 128 + (b & 7) * 16) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          for (int mt = 0; mt < n_mt; ++mt)
            for (int j = 0; j < kKC / 16; ++j)
              umma_bf16(tmem + dcol + mt * B,
                        umma_desc(smem_u32(tA) + mt * 16 * sbo_k64 + j * 256, 128, sbo_k64),
                        umma_desc(smem_u32(tB) + j * 256, 128, sbo_k64), idesc, (c > 0 || j > 0) ? 1u : 0u);
          umma_commit(fbar[s].bar);
        }
        ++fbar[s].issued;
      }
      bar_drain(fbar[0], failed);
      bar_drain(fbar[1], failed);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // partial Z0^T (lane = hidden unit, column = batch index) -> global scratch [b][n]
      {
        float* part = act + G.part[l] + (size_t)rank * B * out0;
        const int span = n_mt * B;
        const int nsplit = min(kColSplit, span / 16), half = span / nsplit;
        for (int cc0 = (warp >> 2) * half; (warp >> 2) < nsplit && cc0 < ((warp >> 2) + 1) * half; cc0 += 16) {
          uint32_t v[16];
          tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + dcol + cc0, v);
          const int mt = cc0 / B, b0 = cc0 % B;
          const int n = mt * 128 + (warp & 3) * 32 + lane;
#pragma unroll
          for (int i = 0; i < 16; ++i) part[(size_t)(b0 + i) * out0 + n] = __uint_as_float(v[i]);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      cluster_sync(clustered);
      // bias + ReLU + bf16 rounding of the columns this CTA feeds into the next layer
      {
        const float* part0 = act + G.part[l];
        const float* bias = work + boff[l];
        const int c_lo = r0[l + 1], c_n = r1[l + 1] - r0[l + 1];
        staged_copy(B * c_n, tid,
                    [&](int e) { const int b = e / c_n, n = c_lo + e % c_n;
                                 float z = bias[n];
                                 for (int r = 0; r < C; ++r) z += part0[((size_t)r * B + b) * out0 + n];
                                 return z; },
                    [&](int e, float z) { act[G.a[l] + (size_t)(e / c_n) * out0 + c_lo + e % c_n] = q_bf16(fmaxf(z, 0.f)); });
        __syncthreads();
      }
    };
    fwd_tc(0, it > 0);

    // ================= forward, layers >= 1 (FMA) =================
    for (int l = 1; l < L; ++l) {
      if (tc_layer[l]) { fwd_tc(l, false); continue; }
      const int N = (int)S.dims[l + 1], Np = up4(N), ldw = Np + 4;
      const int tiles_n = Np / 4, ntile = (B / 4) * tiles_n;
      float acc[kMaxTiles][16];
#pragma unroll
      for (int q = 0; q < kMaxTiles; ++q)
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[q][e] = 0.f;
      for (int c0 = r0[l]; c0 < r1[l]; c0 += kRC) {
        const int rc = min(kRC, r1[l] - c0);
        __syncthreads();
        staged_copy(kRC * B, tid,
                    [&](int e) { const int b = e / kRC, ic = e % kRC;
                                 return ic < rc ? act[G.a[l - 1] + (size_t)b * S.dims[l] + c0 + ic] : 0.f; },
                    [&](int e, float v) { As[(e % kRC) * B + e / kRC] = v; });
        staged_copy(kRC * Np, tid,
                    [&](int e) { const int ic = e / Np, j = e % Np;
                                 return (ic < rc && j < N) ? q_bf16(work[woff[l] + (size_t)(c0 + ic) * N + j]) : 0.f; },
                    [&](int e, float v) { Ws[(e / Np) * ldw + e % Np] = v; });
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxTiles; ++q) {
          const int mt = tid + q * kThreads;
          if (mt < ntile) {
            const int bt = mt / tiles_n, jt = mt % tiles_n;
            for (int ic = 0; ic < rc; ++ic) {
              const float4 a = *reinterpret_cast<const float4*>(As + ic * B + 4 * bt);
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
      {
        float* part = act + G.part[l] + (size_t)rank * B * N;
#pragma unroll
        for (int q = 0; q < kMaxTiles; ++q) {
          const int mt = tid + q * kThreads;
          if (mt < ntile) {
            const int bt = mt / tiles_n, jt = mt % tiles_n;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int n = 4 * jt + j;
                if (n < N) part[(size_t)(4 * bt + i) * N + n] = acc[q][4 * i + j];
              }
          }
        }
      }
      cluster_sync(clustered);
      const float* part0 = act + G.part[l];
      const float* bias = work + boff[l];
      if (l < L - 1) {
        const int c_lo = r0[l + 1], c_n = r1[l + 1] - r0[l + 1];
        staged_copy(B * c_n, tid,
                    [&](int e) { const int b = e / c_n, n = c_lo + e % c_n;
                                 float z = bias[n];
                                 for (int r = 0; r < C; ++r) z += part0[((size_t)r * B + b) * N + n];
                                 return z; },
                    [&](int e, float z) { act[G.a[l] + (size_t)(e / c_n) * N + c_lo + e % c_n] = q_bf16(fmaxf(z, 0.f)); });
        __syncthreads();
      } else {
        staged_copy(B * N, tid,
                    [&](int e) { const int b = e / N, n = e % N;
                                 float z = bias[n];
                                 for (int r = 0; r < C; ++r) z += part0[((size_t)r * B + b) * N + n];
                                 return z; },
                    [&](int e, float z) { zs[(e / N) * 32 + e % N] = z; });
        __syncthreads();
        for (int b = tid; b < B; b += kThreads) {
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
            dzq[b * Np + n] = q_bf16(d);
          }
        }
        __syncthreads();
      }
    }

    // ================= backward + update of a hidden layer l >= 1 on tensor cores =================
    auto bwd_tc = [&](const int l) {
      const int out0 = (int)S.dims[l + 1], Kin = (int)S.dims[l], R0 = r1[l] - r0[l];
      const float* dz0 = act + G.dz[l];          // full dZ_l [B, out], fp32, visible after a cluster barrier
      {
        // dZ_{l-1}[b, i] = relu'(A_{l-1}[b, i]) * sum_j W_l[i, j] bf16(dZ_l)[b, j] for the rows i this CTA owns,
        // from the weights as they are before this iteration's update:
        // D[128 rows x B] = bf16(W_l chunk)[128 x out] . bf16(dZ_l)[B x out]^T
        const uint32_t sbo_ko = (out0 / 8) * 128;
        unsigned char* tW = tiles;
        unsigned char* tD = tiles + 128 * out0 * 2;
        const uint32_t idesc_a = umma_idesc(128, B);
        __syncthreads();
        for (int e = tid; e < B * (out0 / 8); e += kThreads) {
          const int kg = e % (out0 / 8), b = e / (out0 / 8);
          const float4* src = reinterpret_cast<const float4*>(dz0 + (size_t)b * out0 + kg * 8);
          const float4 lo = src[0], hi = src[1];
          uint4 v;
          v.x = pack_bf16(lo.x, lo.y); v.y = pack_bf16(lo.z, lo.w); v.z = pack_bf16(hi.x, hi.y); v.w = pack_bf16(hi.z, hi.w);
          *reinterpret_cast<uint4*>(tD + (b >> 3) * sbo_ko + kg * 128 + (b & 7) * 16) = v;
        }
        for (int c0 = r0[l]; c0 < r1[l]; c0 += kMT) {
          for (int e = tid; e < kMT * (out0 / 8); e += kThreads) {
            const int kg = e % (out0 / 8), i = e / (out0 / 8);
            const float4* src = reinterpret_cast<const float4*>(work + woff[l] + (size_t)(c0 + i) * out0 + kg * 8);
            const float4 lo = src[0], hi = src[1];
            uint4 v;
            v.x = pack_bf16(lo.x, lo.y); v.y = pack_bf16(lo.z, lo.w); v.z = pack_bf16(hi.x, hi.y); v.w = pack_bf16(hi.z, hi.w);
            *reinterpret_cast<uint4*>(tW + (i >> 3) * sbo_ko + kg * 128 + (i & 7) * 16) = v;
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncthreads();
          if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int j = 0; j < out0 / 16; ++j)
              umma_bf16(tmem, umma_desc(smem_u32(tW) + j * 256, 128, sbo_ko),
                        umma_desc(smem_u32(tD) + j * 256, 128, sbo_ko), idesc_a, j > 0 ? 1u : 0u);
            umma_commit(fbar[0].bar);
          }
          ++fbar[0].issued;
          bar_drain(fbar[0], failed);
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          {
            const int nsplit = min(kColSplit, B / 16), half = B / nsplit;
            const int i = c0 + (warp & 3) * 32 + lane;   // lane = row of the chunk, columns = batch index
            for (int b0 = (warp >> 2) * half; (warp >> 2) < nsplit && b0 < ((warp >> 2) + 1) * half; b0 += 16) {
              uint32_t v[16];
              tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + b0, v);
              float a[16];
#pragma unroll
              for (int q = 0; q < 16; ++q) a[q] = act[G.a[l - 1] + (size_t)(b0 + q) * Kin + i];
#pragma unroll
              for (int q = 0; q < 16; ++q)
                act[G.dz[l - 1] + (size_t)(b0 + q) * Kin + i] = a[q] > 0.f ? __uint_as_float(v[q]) : 0.f;
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncthreads();   // the tile and the accumulator are free again
        }
      }
      const int a_bytes = kMT * B * 2;
      unsigned char* tBd = tiles + 2 * a_bytes;  // bf16(dZ0)^T: element (row j, col b)
      const uint32_t idesc = umma_idesc(128, out0);
      __syncthreads();
      for (int e = tid; e < out0 * (B / 8); e += kThreads) {
        const int j = e % out0, bg = e / out0;
        const float* src = dz0 + (size_t)(bg * 8) * out0 + j;
        uint4 v;
        v.x = pack_bf16(src[0], src[out0]);
        v.y = pack_bf16(src[2 * (size_t)out0], src[3 * (size_t)out0]);
        v.z = pack_bf16(src[4 * (size_t)out0], src[5 * (size_t)out0]);
        v.w = pack_bf16(src[6 * (size_t)out0], src[7 * (size_t)out0]);
        *reinterpret_cast<uint4*>(tBd + (j >> 3) * sbo_kB + bg * 128 + (j & 7) * 16) = v;
      }
      const int nch = R0 / kMT;
      auto stage_and_issue = [&](int c) {
        const int s = c & 1, c0 = r0[l] + c * kMT;
        unsigned char* tA = tiles + s * a_bytes;  // the layer's input, transposed: element (row i, col b)
        for (int e = tid; e < kMT * (B / 8); e += kThreads) {
          const int i = e % kMT, bg = e / kMT;
          uint4 v;
          const float* col = act + G.a[l - 1] + (size_t)(bg * 8) * Kin + c0 + i;
          float f[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) f[k] = col[(size_t)k * Kin];
          v.x = pack_bf16(f[0], f[1]); v.y = pack_bf16(f[2], f[3]); v.z = pack_bf16(f[4], f[5]); v.w = pack_bf16(f[6], f[7]);
          *reinterpret_cast<uint4*>(tA + (i >> 3) * sbo_kB + bg * 128 + (i & 7) * 16) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          for (int j = 0; j < B / 16; ++j)
            umma_bf16(tmem + s * 256, umma_desc(smem_u32(tA) + j * 256, 128, sbo_kB),
                      umma_desc(smem_u32(tBd) + j * 256, 128, sbo_kB), idesc, j > 0 ? 1u : 0u);
          umma_commit(bbar[s].bar);
        }
        ++bbar[s].issued;
      };
      if (nch > 0) stage_and_issue(0);
      for (int c = 0; c < nch; ++c) {
        const int s = c & 1, c0 = r0[l] + c * kMT;
        if (c + 1 < nch) stage_and_issue(c + 1);   // its buffer and accumulator were released by chunk c-1
        bar_drain(bbar[s], failed);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // epilogue: a warp owns 32 rows of W0 and half of the columns.  The accumulator
        // block comes out of tensor memory one row per lane; a per-warp transpose through
        // shared memory lets every global access cover 4 rows x 128 contiguous bytes.
        float* tr = trbuf + warp * (32 * kTrLd);
        const int half = out0 / kColSplit;   // 64 or 32 columns per warp
        const int rr = lane >> 3, cg = (lane & 7) * 4;
        for (int j0 = (warp >> 2) * half; j0 < ((warp >> 2) + 1) * half; j0 += 32) {
          uint32_t v[32];
          tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + s * 256 + j0, v);
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<float4*>(tr + lane * kTrLd + 4 * q) =
                make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
          __syncwarp();
          const size_t base = woff[l] + (size_t)(c0 + (warp & 3) * 32 + rr) * out0 + j0 + cg;
          const bool with_u = true;
          float4 w[8], u[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {   // rows rr, rr + 4, ...: independent 16-byte loads in flight
            w[q] = *reinterpret_cast<const float4*>(work + base + (size_t)(4 * q) * out0);
            u[q] = with_u ? *reinterpret_cast<const float4*>(Urow + base + (size_t)(4 * q) * out0)
                          : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 gq = *reinterpret_cast<const float4*>(tr + (4 * q + rr) * kTrLd + cg);
            const float g0 = fmaf(lambda, w[q].x, gq.x), g1 = fmaf(lambda, w[q].y, gq.y);
            const float g2 = fmaf(lambda, w[q].z, gq.z), g3 = fmaf(lambda, w[q].w, gq.w);
            w[q].x = fmaf(-eta, g0, w[q].x); w[q].y = fmaf(-eta, g1, w[q].y); w[q].z = fmaf(-eta, g2, w[q].z); w[q].w = fmaf(-eta, g3, w[q].w);
            u[q].x += g0; u[q].y += g1; u[q].z += g2; u[q].w += g3;
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            *reinterpret_cast<float4*>(work + base + (size_t)(4 * q) * out0) = w[q];
            if (with_u) *reinterpret_cast<float4*>(Urow + base + (size_t)(4 * q) * out0) = u[q];
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      }
      cluster_sync(clustered);
      if (rank == l % C)
        for (int n = tid; n < out0; n += kThreads) {
          float gb = 0.f;
          for (int b = 0; b < B; ++b) gb += dz0[(size_t)b * out0 + n];
          work[boff[l] + n] = fmaf(-eta, gb, work[boff[l] + n]);
          Urow[boff[l] + n] += gb;
        }
      if (l > 1 && !tc_layer[l - 1]) {   // the FMA layer below reads dZ_{l-1} from shared memory
        __syncthreads();
        const int Nm = (int)S.dims[l], Nmp = up4(Nm);
        staged_copy(B * Nmp, tid,
                    [&](int e) { const int b = e / Nmp, n = e % Nmp;
                                 return n < Nm ? act[G.dz[l - 1] + (size_t)b * Nm + n] : 0.f; },
                    [&](int e, float d) { dzs[e] = d; dzq[e] = q_bf16(d); });
        __syncthreads();
      }
    };

    // ========== layer 0: backward + update, fused with the next iteration's forward product ==========
    // The gradient G[128 rows x out0] of a chunk is computed in units of 128 columns, two
    // tensor-memory slots of 128 columns taking turns: the MMAs of unit u + 1 run while unit u
    // is read back and applied to the fp32 master.  A unit's updated weights are what the next
    // iteration's forward pass would read again from HBM, so they go, rounded to bf16, from the
    // registers of the epilogue into one more operand tile, and Z0^T[unit's columns x B] +=
    // bf16(W0_new[chunk rows, unit's columns])^T . X_next[:, chunk rows]^T is issued right away into
    // the forward accumulators (columns kFwdCol...).  Chunk by chunk this is the same sum, in the
    // same order, as the stand-alone forward pass, which only the first iteration of a round runs.
    auto bwd0 = [&]() {
      const int out0 = (int)S.dims[1], R0 = r1[0] - r0[0];
      const float* dz0 = act + G.dz[0];
      const int NH = out0 / 128, nch = R0 / kMT, NU = nch * NH;
      const int a_bytes = kMT * B * 2;
      unsigned char* tBd = tiles + 2 * a_bytes;                 // bf16(dZ0)^T: element (row j, col b)
      unsigned char* tWf = tBd + out0 * B * 2;                  // bf16(W0_new) of one unit: element (row j, col i)
      unsigned char* tXf0 = tWf + 128 * kMT * 2;                // next batch's inputs of a chunk: element (row b, col i)
      unsigned char* tXf1 = smraw + M.x2;                       // ... and of the chunk after it
      const uint32_t idesc_b = umma_idesc(128, 128), idesc_f = umma_idesc(128, B);
      const uint32_t sbo_kM = (kMT / 8) * 128;                  // tiles with K = 128
      __syncthreads();
      for (int e = tid; e < out0 * (B / 8); e += kThreads) {
        const int j = e % out0, bg = e / out0;
        const float* src = dz0 + (size_t)(bg * 8) * out0 + j;
        uint4 v;
        v.x = pack_bf16(src[0], src[out0]);
        v.y = pack_bf16(src[2 * (size_t)out0], src[3 * (size_t)out0]);
        v.z = pack_bf16(src[4 * (size_t)out0], src[5 * (size_t)out0]);
        v.w = pack_bf16(src[6 * (size_t)out0], src[7 * (size_t)out0]);
        *reinterpret_cast<uint4*>(tBd + (j >> 3) * sbo_kB + bg * 128 + (j & 7) * 16) = v;
      }
      auto stage = [&](int c) {   // operand tiles of chunk c; ends with a block barrier
        const int c0 = r0[0] + c * kMT;
        unsigned char* tA = tiles + (c & 1) * a_bytes;   // this batch's inputs, transposed: element (row i, col b)
        for (int e = tid; e < kMT * (B / 8); e += kThreads) {
          const int i = e % kMT, bg = e / kMT;
          const __nv_bfloat16* col = xdata + c0 + i;
          unsigned short q[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) q[k] = __ldg(reinterpret_cast<const unsigned short*>(col + (size_t)idx[bg * 8 + k] * D0));
          uint4 v;
          v.x = q[0] | ((uint32_t)q[1] << 16); v.y = q[2] | ((uint32_t)q[3] << 16);
          v.z = q[4] | ((uint32_t)q[5] << 16); v.w = q[6] | ((uint32_t)q[7] << 16);
          *reinterpret_cast<uint4*>(tA + (i >> 3) * sbo_kB + bg * 128 + (i & 7) * 16) = v;
        }
        if (fuse) {
          unsigned char* tX = (c & 1) ? tXf1 : tXf0;
          for (int e = tid; e < B * (kMT / 8); e += kThreads) {
            const int kg = e % (kMT / 8), b = e / (kMT / 8);
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(xdata + (size_t)idxn[b] * D0 + c0 + kg * 8));
            *reinterpret_cast<uint4*>(tX + (b >> 3) * sbo_kM + kg * 128 + (b & 7) * 16) = v;
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
      };
      auto issue_bwd = [&](int u) {   // thread 0: gradient MMAs of unit u into slot u & 1
        const int c = u / NH, hh = u % NH;
        unsigned char* tA = tiles + (c & 1) * a_bytes;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int j = 0; j < B / 16; ++j)
          umma_bf16(tmem + (u & 1) * 128, umma_desc(smem_u32(tA) + j * 256, 128, sbo_kB),
                    umma_desc(smem_u32(tBd) + hh * 16 * sbo_kB + j * 256, 128, sbo_kB), idesc_b, j > 0 ? 1u : 0u);
        umma_commit(bbar[u & 1].bar);
      };
      if (NU > 0) {
        stage(0);
        if (tid == 0) issue_bwd(0);
        ++bbar[0].issued;
      }
      float* tr = trbuf + warp * (32 * kTrLd);
      const int rr = lane >> 3, cg = (lane & 7) * 4;
      for (int u = 0; u < NU; ++u) {
        const int c = u / NH, hh = u % NH, sl = u & 1, c0 = r0[0] + c * kMT;
        if (u + 1 < NU) {
          // slot (u + 1) & 1 was read back by unit u - 1, before the barrier that ended its turn
          if ((u + 1) % NH == 0) {
            if (fuse) bar_drain(fwbar, failed);   // the forward MMAs that read the input tile being replaced
            stage(c + 1);
          }
          if (tid == 0) issue_bwd(u + 1);
          ++bbar[(u + 1) & 1].issued;
        }
        bar_drain(bbar[sl], failed);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // epilogue: a warp owns 32 rows x 32 columns of the unit.  The accumulator block comes
        // out of tensor memory one row per lane; a per-warp transpose through shared memory
        // lets every global access cover 4 rows x 128 contiguous bytes.
        {
          const int jl = (warp >> 2) * 32;          // first column within the unit
          uint32_t v[32];
          tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + sl * 128 + jl, v);
          __syncwarp();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<float4*>(tr + lane * kTrLd + 4 * q) =
                make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
          __syncwarp();
          const size_t base = woff[0] + (size_t)(c0 + (warp & 3) * 32 + rr) * out0 + hh * 128 + jl + cg;
          float4 w[8], uu[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {   // rows rr, rr + 4, ...: independent 16-byte loads in flight
            w[q] = *reinterpret_cast<const float4*>(work + base + (size_t)(4 * q) * out0);
            uu[q] = kDeriveU0 ? make_float4(0.f, 0.f, 0.f, 0.f)
                              : *reinterpret_cast<const float4*>(Urow + base + (size_t)(4 * q) * out0);
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 gq = *reinterpret_cast<const float4*>(tr + (4 * q + rr) * kTrLd + cg);
            const float g0 = fmaf(lambda, w[q].x, gq.x), g1 = fmaf(lambda, w[q].y, gq.y);
            const float g2 = fmaf(lambda, w[q].z, gq.z), g3 = fmaf(lambda, w[q].w, gq.w);
            w[q].x = fmaf(-eta, g0, w[q].x); w[q].y = fmaf(-eta, g1, w[q].y); w[q].z = fmaf(-eta, g2, w[q].z); w[q].w = fmaf(-eta, g3, w[q].w);
            uu[q].x += g0; uu[q].y += g1; uu[q].z += g2; uu[q].w += g3;
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            *reinterpret_cast<float4*>(work + base + (size_t)(4 * q) * out0) = w[q];
            if (!kDeriveU0) *reinterpret_cast<float4*>(Urow + base + (size_t)(4 * q) * out0) = uu[q];
          }
          if (fuse) {
            // the new weights go back through the transpose buffer: a lane then holds 8 consecutive
            // input rows of one column = one 16-byte entry of the K-major operand tile
            bar_drain(fwbar, failed);   // the previous unit's forward MMAs have read the tile
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 8; ++q) *reinterpret_cast<float4*>(tr + (4 * q + rr) * kTrLd + cg) = w[q];
            __syncwarp();
            const int j = jl + lane;
#pragma unroll
            for (int g8 = 0; g8 < 4; ++g8) {
              float f[8];
#pragma unroll
              for (int r = 0; r < 8; ++r) f[r] = tr[(8 * g8 + r) * kTrLd + lane];
              uint4 pk;
              pk.x = pack_bf16(f[0], f[1]); pk.y = pack_bf16(f[2], f[3]); pk.z = pack_bf16(f[4], f[5]); pk.w = pack_bf16(f[6], f[7]);
              const int kg = (warp & 3) * 4 + g8;
              *reinterpret_cast<uint4*>(tWf + (j >> 3) * sbo_kM + kg * 128 + (j & 7) * 16) = pk;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();   // the slot is free again; the weight tile is complete
        if (fuse) {
          if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int j = 0; j < kMT / 16; ++j)
              umma_bf16(tmem + kFwdCol + hh * B, umma_desc(smem_u32(tWf) + j * 256, 128, sbo_kM),
                        umma_desc(smem_u32((c & 1) ? tXf1 : tXf0) + j * 256, 128, sbo_kM), idesc_f, (c > 0 || j > 0) ? 1u : 0u);
            umma_commit(fwbar.bar);
          }
          ++fwbar.issued;
        }
      }
      bar_drain(fwbar, failed);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      cluster_sync(clustered);
      if (rank == 0)
        for (int n = tid; n < out0; n += kThreads) {
          float gb = 0.f;
          for (int b = 0; b < B; ++b) gb += dz0[(size_t)b * out0 + n];
          work[boff[0] + n] = fmaf(-eta, gb, work[boff[0] + n]);
          Urow[boff[0] + n] += gb;
        }
    };

    // ================= backward + update, layers >= 1 (FMA) =================
    for (int l = L - 1; l >= 1; --l) {
      if (tc_layer[l]) { bwd_tc(l); continue; }
      const int N = (int)S.dims[l + 1], Np = up4(N), ldw = Np + 4;
      const int K = (int)S.dims[l];
      for (int c0 = r0[l]; c0 < r1[l]; c0 += kRC) {
        const int rc = min(kRC, r1[l] - c0);
        __syncthreads();
        staged_copy(kRC * B, tid,
                    [&](int e) { const int b = e / kRC, ic = e % kRC;
                                 return ic < rc ? act[G.a[l - 1] + (size_t)b * K + c0 + ic] : 0.f; },
                    [&](int e, float v) { AsT[e] = v; });
        staged_copy(kRC * Np, tid,
                    [&](int e) { const int ic = e / Np, j = e % Np;
                                 return (ic < rc && j < N) ? q_bf16(work[woff[l] + (size_t)(c0 + ic) * N + j]) : 0.f; },
                    [&](int e, float v) { Ws[(e / Np) * ldw + e % Np] = v; });
        __syncthreads();
        for (int e0 = tid; e0 < B * rc; e0 += 8 * kThreads) {   // eight independent dot products per thread
          float s8[8];
          const float* dp[8];
          const float* wq[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int e = min(e0 + q * kThreads, B * rc - 1);
            s8[q] = 0.f;
            dp[q] = dzq + (e / rc) * Np;
            wq[q] = Ws + (e % rc) * ldw;
          }
          for (int j = 0; j < Np; j += 4) {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 d = *reinterpret_cast<const float4*>(dp[q] + j);
              const float4 w = *reinterpret_cast<const float4*>(wq[q] + j);
              s8[q] = fmaf(d.x, w.x, s8[q]); s8[q] = fmaf(d.y, w.y, s8[q]);
              s8[q] = fmaf(d.z, w.z, s8[q]); s8[q] = fmaf(d.w, w.w, s8[q]);
            }
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int e = e0 + q * kThreads;
            if (e < B * rc) {
              const int b = e / rc, ic = e % rc;
              act[G.dz[l - 1] + (size_t)b * K + c0 + ic] = AsT[b * kRC + ic] > 0.f ? s8[q] : 0.f;
            }
          }
        }
        {
          const int tiles_n = Np / 4, ntile = (kRC / 4) * tiles_n;
          for (int mt = tid; mt < ntile; mt += kThreads) {
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
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const int ic = 4 * it4 + i, n = 4 * jt + j;
                if (ic < rc && n < N) {
                  const size_t o = woff[l] + (size_t)(c0 + ic) * N + n;
                  const float gg = fmaf(lambda, wv[4 * i + j], g[4 * i + j]);
                  work[o] = fmaf(-eta, gg, wv[4 * i + j]);
                  Urow[o] = uv[4 * i + j] + gg;
                }
              }
          }
        }
      }
      cluster_sync(clustered);
      if (rank == l % C)
        for (int n = tid; n < N; n += kThreads) {
          float gb = 0.f;
          for (int b = 0; b < B; ++b) gb += dzs[b * Np + n];
          work[boff[l] + n] = fmaf(-eta, gb, work[boff[l] + n]);
          Urow[boff[l] + n] += gb;
        }
      if (l > 1 && !tc_layer[l - 1]) {
        __syncthreads();
        const int Nm = (int)S.dims[l], Nmp = up4(Nm);
        staged_copy(B * Nmp, tid,
                    [&](int e) { const int b = e / Nmp, n = e % Nmp;
                                 return n < Nm ? act[G.dz[l - 1] + (size_t)b * Nm + n] : 0.f; },
                    [&](int e, float d) { dzs[e] = d; dzq[e] = q_bf16(d); });
        __syncthreads();
      }
    }

    bwd0();
    h += (uint32_t)B;
  }

  // ---- event trigger: publish (c, U_i, i) ----
  cluster_sync(clustered);
  if (kDeriveU0) {   // U_0 = (w_start - w_end) / eta on this CTA's rows of W_0
    const float inv_eta = 1.f / eta;
    const size_t lo = woff[0] + (size_t)r0[0] * S.dims[1], hi = woff[0] + (size_t)r1[0] * S.dims[1];
    for (size_t j = lo + 4 * (size_t)tid; j < hi; j += 4 * kThreads) {   // slices start and end on 16-byte boundaries
      const float4 a = *reinterpret_cast<const float4*>(Urow + j), b = *reinterpret_cast<const float4*>(work + j);
      *reinterpret_cast<float4*>(Urow + j) =
          make_float4((a.x - b.x) * inv_eta, (a.y - b.y) * inv_eta, (a.z - b.z) * inv_eta, (a.w - b.w) * inv_eta);
    }
  }
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
  if (failed && tid == 0 && p.r.status) atomicOr(p.r.status, 1u);
  if (rank == 0 && tid == 0) {
    TriggerRec rec;
    rec.client = t.client; rec.round = t.round; rec.samples_done = h; rec.flags = 1;
    p.r.trig[t.seq] = rec;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

bool mlp_tc_eligible(const MlpShape& s) {
  if (s.precision != 1 || s.n_layers < 2 || s.cluster == 0) return false;
  const uint32_t out0 = s.dims[1], B = s.batch;
  if (out0 != 128 && out0 != 256) return false;
  if (B != 32 && B != 64) return false;
  if (s.dims[0] % (s.cluster * 128)) return false;           // every CTA owns whole 128-row chunks
  for (uint32_t l = 1; l < s.n_layers; ++l)
    if (((B + 3) / 4) * ((s.dims[l + 1] + 3) / 4) > (uint32_t)(kMaxTiles * kThreads)) return false;
  if (s.dims[s.n_layers] > 32) return false;
  return (size_t)make_tc_smem(s).total <= 227 * 1024;
}

cudaError_t launch_mlp_tc_rounds(const MlpLaunch& p, cudaStream_t s) {
  if (p.r.n_tasks == 0) return cudaSuccess;
  // More than half of an SM's shared memory: never two of these CTAs on one SM, so the
  // 512-column tensor-memory allocation of one can never wait on a cluster peer.
  size_t smem = (size_t)make_tc_smem(p.shape).total;
  if (smem < 120 * 1024) smem = 120 * 1024;
  // The shared-memory opt-in is a per-device attribute of the kernel and cheap to set: set it on
  // every launch rather than caching it per process (a second device, or two host threads).
  {
    cudaError_t e = cudaFuncSetAttribute(mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
  return cudaLaunchKernelEx(&cfg, mlp_tc_kernel, p);
}

}  // namespace aet
