// Local-SGD round of one client for the bf16-operand MLP D0 -> 256 -> 128 -> C (C <= 16), minibatch
// 64: one CTA per round-task streams the first layer's fp32 master through the tensor cores once per
// SGD iteration, in a warp-specialised pipeline.
//
// Algorithm 3, MainComputeNode, inner loop with xi a minibatch (mean gradient; w_c -= eta_i g;
// U_i += g).  Rounding points as everywhere in the bf16 path: inputs once at load, W_l on every
// read of the fp32 master, hidden activations after bias + ReLU, dZ_l before the two backward
// products; logits, softmax, bias gradients, master updates in fp32.
//
// Every matrix lives in shared memory exactly once, in its natural orientation, as a K-major
// no-swizzle core-matrix tile (8 rows x 16 bytes); a product that needs the transposed view takes
// the same bytes as an MN-major operand (instruction-descriptor major bit, leading / stride byte
// offsets swapped), so nothing is ever transposed by threads:
//   activations are kept transposed, features on the accumulator's lanes, the batch on its columns:
//   Z0^T[h0, b] += W0[i, h0]^T X[b, i]^T     A = MN-major view of the W0 unit tile (rows i, cols h0), B = X tile (rows b, cols i)
//   Z1^T[h1, b]  = W1[h0, h1]^T A0^T[h0, b]  A = MN-major view of the W1 tile, B = MN-major view of the A0^T tile
//   dW1[h0, h1]  = A0^T[h0, b] dZ1^T[h1, b]^T  A = A0^T tile, B = dZ1^T tile (both K-major)
//   dA0^T[h0, b] = W1[h0, h1] dZ1^T[h1, b]   A = W1 tile, B = MN-major view of the dZ1^T tile
//   G[i, h0]     = X[b, i]^T dZ0^T[h0, b]^T  A = MN-major view of the X tile, B = dZ0^T tile
// so every epilogue thread (one accumulator lane = one row of a weight matrix or one hidden unit)
// reads and writes whole 16-byte pieces of rows: the fp32 master in HBM/L2 row by row, the operand
// tiles without bank-scattered 2-byte stores.
//
// Layer 0 (95 % of the flops) runs as a pipeline over units of 128 input rows x 128 hidden columns:
//   warp 8     issues the products: gradient G of unit u + 1 into one of two tensor-memory slots,
//              then the forward product of the NEXT iteration for unit u from the weights the
//              epilogue has just updated (so W0 is read once per iteration, not twice);
//   warps 0-7  epilogue: the master rows of unit u + 1 are already on their way (register
//              prefetch) while unit u is read back from tensor memory, g = G + lambda W,
//              W -= eta g goes back to the master and, rounded to bf16, into the unit tile; the
//              minibatch rows of the next chunk arrive by cp.async straight into their tiles.
// mbarriers carry every hand-over (slot full / slot free, unit tile ready / free, rows landed);
// every wait is bounded, a wait that runs out flags `status`, stops polling and keeps the counters
// moving so that the CTA still leaves through the tensor-memory release.
// Inside a round the fp32 masters of the two wide layers live in the client's work row in the order
// the epilogues touch them, [block][16-byte piece][row of the block][4 floats], so that the 32 lanes of
// a warp - one matrix row each, as tensor memory hands the accumulator out - read and write 512
// contiguous bytes per instruction (row by row a warp instruction would touch 32 different lines, half
// a sector each, and the load/store unit, not HBM, would set the pace: measured 14 K cycles per unit).
// The start of the round writes that order from the snapshot, the trigger reads it back.
// When the launch has SMs to spare (two per round-task), a round-task runs on a cluster of two CTAs:
// each takes one half of the hidden units of layer 0 - its half of every chunk of W0 (so each streams
// half of the master), its rows of W1 - and everything narrower is computed by both.  What crosses
// between them goes through distributed shared memory: the bf16 activations A0^T of the own hidden
// units into the peer's copy after the forward epilogue, the updated bf16 rows of W1 into the peer's W1
// tile; two hardware cluster barriers per iteration order these pushes against the products that read
// them (and a last one keeps a CTA alive until its peer has stopped writing to it).
// The update sums of the two wide layers are not accumulated entry by entry: their rows of U hold
// w_start during the round and become (w_start - w_end) / eta at the trigger (w -= eta g and U += g
// in the same step, eta constant within the round); W2 and the biases accumulate theirs explicitly.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"

namespace aet {
namespace {

constexpr int kH0 = 256, kH1 = 128, kB = 64, kCh = 128;   // widths, minibatch, rows of a chunk
constexpr int kEWarps = 8, kEThreads = kEWarps * 32, kSThreads = kEThreads + 32;   // epilogue warps + the issuing warp
constexpr int kMaxC = 16;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColZ0 = 0, kColG = 128, kColZ1 = 128, kColdW1 = 128, kColdA0 = 384;
constexpr uint32_t kWaitLimit = 1u << 22;

// shared memory map (bytes)
constexpr int kOffW1 = 0;                          // W1 tile, rows h0 (256), cols h1 (128), bf16: 64 KB
constexpr int kOffdZ0 = kOffW1 + kH0 * kH1 * 2;    // dZ0^T tile, rows h0 (256), cols b (64): 32 KB; a CTA of a pair keeps its own
constexpr int kOffA0peer = kOffdZ0 + 128 * kB * 2; //   128 rows there and, behind them, the peer's half of A0^T (16 KB)
constexpr int kOffX = kOffdZ0 + kH0 * kB * 2;      // 4 minibatch-row tiles, rows b (64), cols i (128): cur[2], next[2], 16 KB each;
                                                   // outside the layer-0 pipeline the first 32 KB hold the A0^T tile (two halves of
                                                   // 128 rows; a CTA of a pair keeps only its own half here)
constexpr int kOffA0 = kOffX;
constexpr int kOffWn = kOffX + 4 * kB * kCh * 2;   // unit tile, rows i (128), cols h0 (128), bf16: 32 KB; outside the pipeline:
constexpr int kOffA1 = kOffWn;                     //   A1^T as plain bf16 [h1][b] (16 KB)
constexpr int kOffdZ1 = kOffWn + kH1 * kB * 2;     //   dZ1^T tile, rows h1 (128), cols b (64) (16 KB)
// while the class layer runs, the (not yet written) dZ0^T area holds bf16(W2) as this iteration's products read
// it, and dZ2 rounded to bf16 as [c][b] (conflict-free where lanes differ in b)
constexpr int kOffW2q = kOffdZ0;
constexpr int kOffdZ2T = kOffdZ0 + kH1 * kMaxC * 4;
constexpr int kOffSmall = kOffWn + kCh * 128 * 2;
struct Small {
  float W2[kH1 * kMaxC], UW2[kH1 * kMaxC];
  float b0[kH0], Ub0[kH0], b1[kH1], Ub1[kH1], b2[kMaxC], Ub2[kMaxC];
  float logits[kB * kMaxC], dz2[kB * kMaxC], dz2q[kB * kMaxC];   // [b][c]
  float gb0[2][128];                                               // bias gradient of layer 0, per half of the batch (pairs only)
  int idx[2][kB], ylab[kB];
  uint64_t bar_mma, g_full[2], g_free[2], wn_ready, wn_free, x_ready[2];
  uint32_t tmem_base, failed;
};
constexpr int kSmemBytes = kOffSmall + (int)sizeof(Small);
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// byte offset of element (r, c) of a bf16 tile with `cols` columns
__device__ __forceinline__ int tile_off(int r, int c, int cols) { return (r >> 3) * (cols >> 3) * 128 + (c >> 3) * 128 + (r & 7) * 16 + (c & 7) * 2; }
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// K-major view of a tile with `cols` columns (operand rows = tile rows): row0 and k0 multiples of 8
__device__ __forceinline__ uint64_t view_k(uint32_t base, int cols, int row0, int k0) {
  const uint32_t sr = (uint32_t)(cols >> 3) * 128u;
  return umma_desc(base + (uint32_t)(row0 >> 3) * sr + (uint32_t)(k0 >> 3) * 128u, 128u, sr);
}
// MN-major view (operand M/N index = tile column, K = tile row): LBO = stride of an 8-row group, SBO = of an 8-column group
__device__ __forceinline__ uint64_t view_mn(uint32_t base, int cols, int mn0, int k0) {
  const uint32_t sr = (uint32_t)(cols >> 3) * 128u;
  return umma_desc(base + (uint32_t)(k0 >> 3) * sr + (uint32_t)(mn0 >> 3) * 128u, sr, 128u);
}
__device__ __forceinline__ uint32_t idesc_bf16(int M, int N, int a_mn, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float q_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }
// Work-row order of the wide layers' masters (in floats, relative to the layer's first weight).
// W0 [D0, 256]: block = (chunk of 128 rows, half of the columns, half of that) = 128 rows x 64 columns
__device__ __forceinline__ size_t w0_block(int c, int hh, int half) { return (size_t)(((c * 2 + hh) * 2 + half) * 16) * 512; }
// W1 [256, 128]: block = (half of the rows, group of 32 columns) = 128 rows x 32 columns
__device__ __forceinline__ size_t w1_block(int tl, int g32) { return (size_t)((tl * 4 + g32) * 8) * 512; }
// within a block: 16-byte piece k of row r sits at (k * 128 + r) * 4
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}

// distributed shared memory of the CTA pair
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t saddr, uint32_t peer) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(peer));
  return r;
}
__device__ __forceinline__ void st_peer16(uint32_t addr, const uint4 v) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Bounded wait for the completion number `count` (0-based) of an mbarrier.  After a timeout nothing polls any more.
__device__ __forceinline__ void mbar_wait_n(uint64_t* bar, uint32_t count, bool& failed) {
  const uint32_t parity = count & 1u;
  bool ok = failed;
  for (uint32_t i = 0; i < kWaitLimit && !ok; ++i) {
    uint32_t p;
    asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                 : "=r"(p) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    ok = p != 0;
  }
  if (!ok) failed = true;
}

// NR = CTAs per round-task (1, or 2 as a cluster that splits the hidden units of layer 0)
template <int NR>
__global__ void __launch_bounds__(kSThreads, 1) mlp_stream_kernel(MlpLaunch p) {
  extern __shared__ __align__(1024) unsigned char sm[];
  Small& S = *reinterpret_cast<Small*>(sm + kOffSmall);
  constexpr int UPC = 2 / NR;   // units of a chunk this CTA works through
  const int rank = NR == 2 ? (int)cluster_rank() : 0;
  const uint32_t peer = (uint32_t)(rank ^ 1);
  const TaskDesc t = p.r.tasks[p.r.task_begin + blockIdx.x / NR];
  if (!debug_task_ok(p.r, t)) return;   // debug checks only: rows and slots in range, else flag and skip (both CTAs of a pair alike)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool ewarp = warp < kEWarps;
  const int D0 = (int)p.shape.dims[0], C = (int)p.shape.dims[3];
  const int nch = D0 / kCh, NU = UPC * nch;   // chunks of 128 input rows; units = chunk x half of the hidden columns
  const size_t oW0 = 0, ob0 = (size_t)D0 * kH0, oW1 = ob0 + kH0, ob1 = oW1 + (size_t)kH0 * kH1, oW2 = ob1 + kH1,
               ob2 = oW2 + (size_t)kH1 * C;
  float* work = p.work + (size_t)t.client * p.r.stride;
  float* Urow = p.r.U + (size_t)t.u_row * p.r.stride;
  const ClientData cd = p.r.clients[t.client];
  const __nv_bfloat16* xdata = reinterpret_cast<const __nv_bfloat16*>(cd.x);
  const uint64_t key = p.r.sample_keys[t.client];
  const float eta = t.eta, lambda = p.r.l2;
  const uint32_t sW1 = smem_u32(sm + kOffW1), sdZ0 = smem_u32(sm + kOffdZ0), sWn = smem_u32(sm + kOffWn),
                 sdZ1 = smem_u32(sm + kOffdZ1), sX = smem_u32(sm + kOffX);
  // A0^T, rows [128 tl, 128 tl + 128): a pair keeps the own half where a single CTA keeps its first, the peer's apart
  auto a0_half = [&](int tl) { return NR == 1 ? kOffA0 + tl * 128 * kB * 2 : (tl == rank ? kOffA0 : kOffA0peer); };
  auto unit_hh = [&](int u) { return NR == 1 ? (u & 1) : rank; };

  // ---- barriers and tensor memory ----
  if (tid == 0) {
    auto init = [](uint64_t* b, uint32_t n) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(n)); };
    init(&S.bar_mma, 1);
    init(&S.g_full[0], 1); init(&S.g_full[1], 1);
    init(&S.g_free[0], kEWarps); init(&S.g_free[1], kEWarps);
    init(&S.wn_ready, kEWarps); init(&S.wn_free, 1);
    init(&S.x_ready[0], kEWarps); init(&S.x_ready[1], kEWarps);
    S.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&S.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = S.tmem_base;
  const uint32_t tq = tmem + ((uint32_t)((warp & 3) * 32) << 16);   // this warp's quarter of the lanes
  bool failed = false;
  // completions seen so far: the counters run on from iteration to iteration
  uint32_t n_mma = 0, n_gfull[2] = {0, 0}, n_gfree[2] = {0, 0}, n_wnready = 0, n_wnfree = 0, n_xready[2] = {0, 0};

  // ---- start model: snapshot minus own update sums still in flight; rows of U of the wide layers keep w_start ----
  {
    const float* snap = p.r.snaps + (size_t)t.snap_slot * p.r.stride;
    // Eight 16-byte pieces per thread and trip: all loads of a trip (snapshot, then each sum in flight) are issued
    // before its first store, so that a thread has eight lines on their way instead of one load - store chain
    // (the compiler cannot move a load above a store here: the arrays may alias for all it knows).
    constexpr int kTrip = 8;
    // `where(e4, j, d4)` maps the e4-th piece of this CTA's share to its natural float index j and its work-row piece d4
    auto start_range = [&](size_t total, size_t o_layer, auto where) {
      for (size_t base = tid; base < total; base += (size_t)kTrip * kSThreads) {
        float4 w[kTrip];
        size_t jj[kTrip], dd[kTrip];
#pragma unroll
        for (int q = 0; q < kTrip; ++q) {
          const size_t e4 = base + (size_t)q * kSThreads;
          where(e4 < total ? e4 : 0, jj[q], dd[q]);
          w[q] = *reinterpret_cast<const float4*>(snap + jj[q]);
        }
        for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
          const InflightRef ref = p.r.inflight[t.inflight_off + f];
          const float* urow = p.r.U + (size_t)ref.row * p.r.stride;
          float4 u[kTrip];
#pragma unroll
          for (int q = 0; q < kTrip; ++q) u[q] = *reinterpret_cast<const float4*>(urow + jj[q]);
#pragma unroll
          for (int q = 0; q < kTrip; ++q) {
            w[q].x = fmaf(-ref.eta, u[q].x, w[q].x); w[q].y = fmaf(-ref.eta, u[q].y, w[q].y);
            w[q].z = fmaf(-ref.eta, u[q].z, w[q].z); w[q].w = fmaf(-ref.eta, u[q].w, w[q].w);
          }
        }
#pragma unroll
        for (int q = 0; q < kTrip; ++q)
          if (base + (size_t)q * kSThreads < total) {
            *reinterpret_cast<float4*>(work + o_layer + 4 * dd[q]) = w[q];
            *reinterpret_cast<float4*>(Urow + jj[q]) = w[q];
          }
      }
    };
    // W0 and W1 into work-row order.  The walk is in the natural order (a warp takes 512 contiguous bytes of a row:
    // whole lines of the snapshot, of the sums in flight and of U), the work row takes the scattered 16-byte stores;
    // of a pair, each CTA the columns (W0) or rows (W1) it will own.
    constexpr int kColQ = kH0 / 4 / NR;   // float4 columns of W0 a CTA owns
    start_range((size_t)D0 * kColQ, oW0, [&](size_t e4, size_t& j, size_t& d4) {
      const int i = (int)(e4 / kColQ), q = (int)(e4 % kColQ) + (NR == 2 ? rank * kColQ : 0);   // row, float4 column
      const int c = i >> 7, r = i & 127, hh = q >> 5, half = (q >> 4) & 1, k = q & 15;
      d4 = ((size_t)((c * 2 + hh) * 2 + half) << 11) + ((size_t)k << 7) + r;
      j = oW0 + (size_t)i * kH0 + 4 * q;
    });
    start_range((size_t)kH0 * kH1 / 4 / NR, oW1, [&](size_t e4, size_t& j, size_t& d4) {
      const int i = (int)(e4 / (kH1 / 4)) + (NR == 2 ? rank * 128 : 0), q = (int)(e4 % (kH1 / 4));
      const int tl = i >> 7, r = i & 127, g32 = q >> 3, k = q & 7;
      d4 = ((size_t)(tl * 4 + g32) << 10) + ((size_t)k << 7) + r;
      j = oW1 + (size_t)i * kH1 + 4 * q;
    });
    // the narrow rest stays in shared memory for the round (in both CTAs of a pair)
    for (int j = tid; j < kH0 + kH1 + kH1 * C + C; j += kSThreads) {
      const size_t g = j < kH0 ? ob0 + j : (j < kH0 + kH1 ? ob1 + (j - kH0) : oW2 + (j - kH0 - kH1));
      float w = snap[g];
      for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
        const InflightRef ref = p.r.inflight[t.inflight_off + f];
        w = fmaf(-ref.eta, p.r.U[(size_t)ref.row * p.r.stride + g], w);
      }
      if (g < oW1) { S.b0[g - ob0] = w; S.Ub0[g - ob0] = 0.f; }
      else if (g < oW2) { S.b1[g - ob1] = w; S.Ub1[g - ob1] = 0.f; }
      else if (g < ob2) { S.W2[g - oW2] = w; S.UW2[g - oW2] = 0.f; }
      else { S.b2[g - ob2] = w; S.Ub2[g - ob2] = 0.f; }
    }
  }
  if (NR == 2) cluster_sync(); else __syncthreads();   // the peer's half of the W1 master is in place too
  // W1 tile from the master (rows h0, cols h1)
  for (int e = tid; e < kH0 * (kH1 / 8); e += kSThreads) {
    const int r = e / (kH1 / 8), cg = e % (kH1 / 8);
    const float* blk = work + oW1 + w1_block(r >> 7, cg >> 2);
    const int k = (cg & 3) * 2;
    const float4 lo = *reinterpret_cast<const float4*>(blk + (k * 128 + (r & 127)) * 4);
    const float4 hi = *reinterpret_cast<const float4*>(blk + ((k + 1) * 128 + (r & 127)) * 4);
    uint4 v;
    v.x = pack_bf16(lo.x, lo.y); v.y = pack_bf16(lo.z, lo.w); v.z = pack_bf16(hi.x, hi.y); v.w = pack_bf16(hi.z, hi.w);
    *reinterpret_cast<uint4*>(sm + kOffW1 + tile_off(r, cg * 8, kH1)) = v;
  }
  __syncthreads();

  // minibatch rows of chunk c into a tile (rows b, cols i): 16-byte pieces straight from HBM by cp.async
  auto load_x_tile = [&](unsigned char* tile, const int* idx, int c) {
    for (int e = tid; e < kB * (kCh / 8); e += kEThreads) {
      const int b = e / (kCh / 8), kg = e % (kCh / 8);
      cp_async16(tile + tile_off(b, kg * 8, kCh), xdata + (size_t)idx[b] * D0 + (size_t)c * kCh + kg * 8);
    }
  };

  for (uint32_t it = 0; it < t.steps; ++it) {
    int* idx = S.idx[it & 1];
    int* idxn = S.idx[(it + 1) & 1];
    const bool fuse = it + 1 < t.steps;
    for (int b = tid; b < kB; b += kSThreads) {
      if (it == 0) idx[b] = (int)sample_index(draw(key, t.sample_ctr0 + b), cd.n);
      if (fuse) idxn[b] = (int)sample_index(draw(key, t.sample_ctr0 + (uint64_t)(it + 1) * kB + b), cd.n);
    }
    __syncthreads();
    if (tid < kB) S.ylab[tid] = __ldg(cd.y + idx[tid]);

    // ===== first iteration of a round only: the forward product of layer 0 as a pass of its own =====
    if (it == 0) {
      for (int u = 0; u < NU; ++u) {
        const int c = u / UPC, hh = unit_hh(u);
        if (ewarp) {
          if (u % UPC == 0) load_x_tile(sm + kOffX + 2 * kB * kCh * 2, idx, c);     // into next[0]
          const int q = warp & 3, half = warp >> 2;
          const int r = 32 * q + lane;
          const float* src = work + oW0 + w0_block(c, hh, half) + r * 4;
#pragma unroll
          for (int g8 = 0; g8 < 8; ++g8) {
            const float4 lo = *reinterpret_cast<const float4*>(src + (2 * g8) * 512), hi = *reinterpret_cast<const float4*>(src + (2 * g8 + 1) * 512);
            uint4 v;
            v.x = pack_bf16(lo.x, lo.y); v.y = pack_bf16(lo.z, lo.w); v.z = pack_bf16(hi.x, hi.y); v.w = pack_bf16(hi.z, hi.w);
            *reinterpret_cast<uint4*>(sm + kOffWn + tile_off(r, half * 64 + g8 * 8, 128)) = v;
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncthreads();
        if (tid == kEThreads) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t id = idesc_bf16(128, kB, 1, 0);
          for (int ks = 0; ks < kCh / 16; ++ks)
            umma_bf16(tmem + kColZ0 + (NR == 1 ? 64 * hh : 0), view_mn(sWn, 128, 0, ks * 16), view_k(sX + 2 * kB * kCh * 2, kCh, 0, ks * 16), id,
                      (c > 0 || ks > 0) ? 1u : 0u);
          umma_commit(&S.bar_mma);
        }
        mbar_wait_n(&S.bar_mma, n_mma++, failed);
        __syncthreads();   // the tiles are free again
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }

    // ===== Z0 epilogue: A0^T = bf16(relu(Z0^T + b0)); a pair: own hidden units, each warp half of the batch, and a copy to the peer =====
    if (ewarp) {
      const int q = warp & 3, wh = warp >> 2;
      const int tl = NR == 1 ? wh : rank;
      const int lr = 32 * q + lane;
      const float bias = S.b0[128 * tl + lr];
      const int a0off = a0_half(tl);
      const uint32_t remote = NR == 2 ? peer_addr(smem_u32(sm + kOffA0peer), peer) : 0u;
#pragma unroll
      for (int hq = 0; hq < UPC; ++hq) {
        const int hb = NR == 1 ? hq : wh;   // which 32 columns of the batch
        uint32_t v[32];
        tmem_ld32(tq + kColZ0 + (NR == 1 ? 64 * tl : 0) + 32 * hb, v);
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          uint4 o;
          float a[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) a[k] = fmaxf(__uint_as_float(v[g8 * 8 + k]) + bias, 0.f);
          o.x = pack_bf16(a[0], a[1]); o.y = pack_bf16(a[2], a[3]); o.z = pack_bf16(a[4], a[5]); o.w = pack_bf16(a[6], a[7]);
          const int off = tile_off(lr, 32 * hb + g8 * 8, kB);
          *reinterpret_cast<uint4*>(sm + a0off + off) = o;
          if (NR == 2) st_peer16(remote + (uint32_t)off, o);
        }
      }
      asm volatile("fence.proxy.async;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (NR == 2) cluster_sync(); else __syncthreads();   // pair: both halves of A0^T are in both CTAs

    // ===== layer 1 forward: Z1^T[h1, b] = W1^T A0^T =====
    if (tid == kEThreads) {
      asm volatile("fence.proxy.async;" ::: "memory");
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t id = idesc_bf16(128, kB, 1, 1);
      for (int ks = 0; ks < kH0 / 16; ++ks)
        umma_bf16(tmem + kColZ1, view_mn(sW1, kH1, 0, ks * 16), view_mn(smem_u32(sm + a0_half(ks >> 3)), kB, 0, (ks & 7) * 16), id, ks > 0 ? 1u : 0u);
      umma_commit(&S.bar_mma);
    }
    mbar_wait_n(&S.bar_mma, n_mma++, failed);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp < 4) {   // A1^T = bf16(relu(Z1^T + b1)) as plain [h1][b]
      const int h1 = 32 * warp + lane;
      const float bias = S.b1[h1];
#pragma unroll
      for (int hb = 0; hb < 2; ++hb) {
        uint32_t v[32];
        tmem_ld32(tq + kColZ1 + 32 * hb, v);
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          uint4 o;
          float a[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) a[k] = fmaxf(__uint_as_float(v[g8 * 8 + k]) + bias, 0.f);
          o.x = pack_bf16(a[0], a[1]); o.y = pack_bf16(a[2], a[3]); o.z = pack_bf16(a[4], a[5]); o.w = pack_bf16(a[6], a[7]);
          *reinterpret_cast<uint4*>(sm + kOffA1 + (h1 * kB + 32 * hb + g8 * 8) * 2) = o;
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();

    // ===== class layer forward, softmax cross-entropy =====
    const __nv_bfloat16* A1 = reinterpret_cast<const __nv_bfloat16*>(sm + kOffA1);
    float* W2q = reinterpret_cast<float*>(sm + kOffW2q);
    float* dz2qT = reinterpret_cast<float*>(sm + kOffdZ2T);
    for (int e = tid; e < kH1 * C; e += kSThreads) W2q[e] = q_bf16(S.W2[e]);
    __syncthreads();
    for (int e = tid; e < kB * C; e += kSThreads) {
      const int b = e / C, c = e % C;
      float z0 = S.b2[c], z1 = 0.f, z2 = 0.f, z3 = 0.f;   // four chains in flight: the loads and converts have latency
#pragma unroll 4
      for (int h = 0; h < kH1; h += 4) {
        z0 = fmaf(__bfloat162float(A1[h * kB + b]), W2q[h * C + c], z0);
        z1 = fmaf(__bfloat162float(A1[(h + 1) * kB + b]), W2q[(h + 1) * C + c], z1);
        z2 = fmaf(__bfloat162float(A1[(h + 2) * kB + b]), W2q[(h + 2) * C + c], z2);
        z3 = fmaf(__bfloat162float(A1[(h + 3) * kB + b]), W2q[(h + 3) * C + c], z3);
      }
      S.logits[b * kMaxC + c] = (z0 + z1) + (z2 + z3);
    }
    __syncthreads();
    if (tid < kB) {
      const float* z = S.logits + tid * kMaxC;
      float m = -INFINITY;
      for (int c = 0; c < C; ++c) m = fmaxf(m, z[c]);
      float sum = 0.f;
      for (int c = 0; c < C; ++c) sum += __expf(z[c] - m);
      const float inv = 1.f / sum, invB = 1.f / (float)kB;
      const int y = S.ylab[tid];
      for (int c = 0; c < kMaxC; ++c) {
        const float d = c < C ? (__expf(z[c] - m) * inv - (c == y ? 1.f : 0.f)) * invB : 0.f;
        S.dz2[tid * kMaxC + c] = d;
        S.dz2q[tid * kMaxC + c] = q_bf16(d);
        dz2qT[c * kB + tid] = q_bf16(d);
      }
    }
    __syncthreads();
    // ===== class layer backward: dZ1^T = relu'(A1^T) * (W2 dZ2^T) from the old W2; its bias gradient in fp32 =====
    for (int e = tid; e < kH1 * (kB / 8); e += kSThreads) {
      const int h = e >> 3, bc = e & 7;
      float wq[kMaxC];
#pragma unroll
      for (int c = 0; c < kMaxC; ++c) wq[c] = c < C ? W2q[h * C + c] : 0.f;
      float d[8], part = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int b = bc * 8 + k;
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxC; ++c) s = fmaf(dz2qT[c * kB + b], wq[c], s);   // columns >= C hold zeros
        d[k] = __bfloat162float(A1[h * kB + b]) > 0.f ? s : 0.f;
        part += d[k];
      }
      uint4 o;
      o.x = pack_bf16(d[0], d[1]); o.y = pack_bf16(d[2], d[3]); o.z = pack_bf16(d[4], d[5]); o.w = pack_bf16(d[6], d[7]);
      *reinterpret_cast<uint4*>(sm + kOffdZ1 + tile_off(h, bc * 8, kB)) = o;
      // the eight pieces of a hidden unit sit in eight neighbouring lanes
      part += __shfl_xor_sync(0xffffffffu, part, 1);
      part += __shfl_xor_sync(0xffffffffu, part, 2);
      part += __shfl_xor_sync(0xffffffffu, part, 4);
      if (bc == 0) { S.b1[h] = fmaf(-eta, part, S.b1[h]); S.Ub1[h] += part; }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // pair: from here on the peer may overwrite its rows of this CTA's W1 tile and, in the next iteration, its half
    // of A0^T; both were last read by the forward product of layer 1 above, which both CTAs have seen complete
    if (NR == 2) cluster_sync(); else __syncthreads();
    // ===== layer 1 backward on tensor cores (old W1): dA0^T first, then dW1; a pair: the own 128 hidden units only =====
    if (tid == kEThreads) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t ida = idesc_bf16(128, kB, 0, 1), idw = idesc_bf16(128, kH1, 0, 0);
      for (int tl = NR == 1 ? 0 : rank; tl < (NR == 1 ? 2 : rank + 1); ++tl)
        for (int ks = 0; ks < kH1 / 16; ++ks)
          umma_bf16(tmem + kColdA0 + (NR == 1 ? 64 * tl : 0), view_k(sW1, kH1, 128 * tl, ks * 16), view_mn(sdZ1, kB, 0, ks * 16), ida, ks > 0 ? 1u : 0u);
      for (int tl = NR == 1 ? 0 : rank; tl < (NR == 1 ? 2 : rank + 1); ++tl)
        for (int ks = 0; ks < kB / 16; ++ks)
          umma_bf16(tmem + kColdW1 + (NR == 1 ? 128 * tl : 0), view_k(smem_u32(sm + a0_half(tl)), kB, 0, ks * 16), view_k(sdZ1, kB, 0, ks * 16), idw, ks > 0 ? 1u : 0u);
      umma_commit(&S.bar_mma);
    }
    // meanwhile: the class layer's own update (its products above used the old values)
    for (int e = tid; e < kH1 * C + C; e += kSThreads) {
      if (e < kH1 * C) {
        const int h = e / C, c = e % C;
        float g0 = 0.f, g1 = 0.f, g2 = 0.f, g3 = 0.f;
#pragma unroll 4
        for (int b = 0; b < kB; b += 4) {
          g0 = fmaf(__bfloat162float(A1[h * kB + b]), S.dz2q[b * kMaxC + c], g0);
          g1 = fmaf(__bfloat162float(A1[h * kB + b + 1]), S.dz2q[(b + 1) * kMaxC + c], g1);
          g2 = fmaf(__bfloat162float(A1[h * kB + b + 2]), S.dz2q[(b + 2) * kMaxC + c], g2);
          g3 = fmaf(__bfloat162float(A1[h * kB + b + 3]), S.dz2q[(b + 3) * kMaxC + c], g3);
        }
        float g = (g0 + g1) + (g2 + g3);
        const float w = S.W2[e];
        g = fmaf(lambda, w, g);
        S.W2[e] = fmaf(-eta, g, w);
        S.UW2[e] += g;
      } else {
        const int c = e - kH1 * C;
        float g = 0.f;
        for (int b = 0; b < kB; ++b) g += S.dz2[b * kMaxC + c];
        S.b2[c] = fmaf(-eta, g, S.b2[c]);
        S.Ub2[c] += g;
      }
    }
    mbar_wait_n(&S.bar_mma, n_mma++, failed);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ewarp) {
      const int q = warp & 3, wh = warp >> 2;
      const int tl = NR == 1 ? wh : rank;
      const int lr = 32 * q + lane, h0 = 128 * tl + lr;
      const int a0off = a0_half(tl), dz0row = NR == 1 ? h0 : lr;
      // dZ0^T = relu'(A0^T) * dA0^T; bias gradient of layer 0 in fp32 (a thread sees its unit's whole batch, in a pair half of it)
      float gb = 0.f;
#pragma unroll
      for (int hq = 0; hq < UPC; ++hq) {
        const int hb = NR == 1 ? hq : wh;
        uint32_t v[32];
        tmem_ld32(tq + kColdA0 + (NR == 1 ? 64 * tl : 0) + 32 * hb, v);
#pragma unroll
        for (int g8 = 0; g8 < 4; ++g8) {
          const uint4 a = *reinterpret_cast<const uint4*>(sm + a0off + tile_off(lr, 32 * hb + g8 * 8, kB));
          const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
          float d[8];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            d[2 * k] = bf_lo(aw[k]) > 0.f ? __uint_as_float(v[g8 * 8 + 2 * k]) : 0.f;
            d[2 * k + 1] = bf_hi(aw[k]) > 0.f ? __uint_as_float(v[g8 * 8 + 2 * k + 1]) : 0.f;
            gb += d[2 * k] + d[2 * k + 1];
          }
          uint4 o;
          o.x = pack_bf16(d[0], d[1]); o.y = pack_bf16(d[2], d[3]); o.z = pack_bf16(d[4], d[5]); o.w = pack_bf16(d[6], d[7]);
          *reinterpret_cast<uint4*>(sm + kOffdZ0 + tile_off(dz0row, 32 * hb + g8 * 8, kB)) = o;
        }
      }
      if (NR == 1) {
        S.b0[h0] = fmaf(-eta, gb, S.b0[h0]);
        S.Ub0[h0] += gb;
      } else {
        S.gb0[wh][lr] = gb;   // summed over the two halves of the batch behind the barrier below
      }
      // dW1 epilogue: row h0 of the master, new bf16 values into the W1 tile (a pair: and into the peer's)
      const uint32_t remote = NR == 2 ? peer_addr(sW1, peer) : 0u;
#pragma unroll 1
      for (int gq = 0; gq < 2 * UPC; ++gq) {
        const int g32 = NR == 1 ? gq : 2 * wh + gq;
        float* wrow = work + oW1 + w1_block(tl, g32) + lr * 4;
        uint32_t v[32];
        tmem_ld32(tq + kColdW1 + (NR == 1 ? 128 * tl : 0) + 32 * g32, v);
        float4 w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) w[k] = *reinterpret_cast<const float4*>(wrow + k * 512);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          w[k].x = fmaf(-eta, fmaf(lambda, w[k].x, __uint_as_float(v[4 * k])), w[k].x);
          w[k].y = fmaf(-eta, fmaf(lambda, w[k].y, __uint_as_float(v[4 * k + 1])), w[k].y);
          w[k].z = fmaf(-eta, fmaf(lambda, w[k].z, __uint_as_float(v[4 * k + 2])), w[k].z);
          w[k].w = fmaf(-eta, fmaf(lambda, w[k].w, __uint_as_float(v[4 * k + 3])), w[k].w);
          *reinterpret_cast<float4*>(wrow + k * 512) = w[k];
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          uint4 o;
          o.x = pack_bf16(w[2 * k].x, w[2 * k].y); o.y = pack_bf16(w[2 * k].z, w[2 * k].w);
          o.z = pack_bf16(w[2 * k + 1].x, w[2 * k + 1].y); o.w = pack_bf16(w[2 * k + 1].z, w[2 * k + 1].w);
          const int off = tile_off(h0, 32 * g32 + 8 * k, kH1);
          *reinterpret_cast<uint4*>(sm + kOffW1 + off) = o;
          if (NR == 2) st_peer16(remote + (uint32_t)off, o);
        }
      }
      asm volatile("fence.proxy.async;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();   // dZ0^T and the new W1 tile are complete; the A0^T area becomes minibatch-row tiles
    if (NR == 2 && tid < 128) {
      const float gb = S.gb0[0][tid] + S.gb0[1][tid];
      S.b0[128 * rank + tid] = fmaf(-eta, gb, S.b0[128 * rank + tid]);
      S.Ub0[128 * rank + tid] += gb;
    }

    // ===== layer 0: gradient, master update and the next iteration's forward product, unit by unit =====
    if (ewarp) {
      const int q = warp & 3, half = warp >> 2;
      const int r = 32 * q + lane;                       // row of the unit this thread owns
      // rows of chunks 0 and 1 of this minibatch (gradient products), of chunk 0 of the next one (forward product)
      load_x_tile(sm + kOffX, idx, 0);
      if (nch > 1) load_x_tile(sm + kOffX + kB * kCh * 2, idx, 1);
      if (fuse) load_x_tile(sm + kOffX + 2 * kB * kCh * 2, idxn, 0);
      asm volatile("cp.async.wait_all;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&S.x_ready[0]);
        if (nch > 1) mbar_arrive(&S.x_ready[1]);
      }
      float4 wn[16];
      {
        const float* src = work + oW0 + w0_block(0, unit_hh(0), half) + r * 4;
#pragma unroll
        for (int k = 0; k < 16; ++k) wn[k] = *reinterpret_cast<const float4*>(src + k * 512);
      }
      for (int u = 0; u < NU; ++u) {
        const int c = u / UPC, hh = unit_hh(u), sl = u & 1;
        const bool first = u % UPC == 0, last = u % UPC == UPC - 1, more = c + 1 < nch;
        float4 w[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k] = wn[k];
        float* dst = work + oW0 + w0_block(c, hh, half) + r * 4;
        // The gradient of this unit was issued a unit ago; taking its barrier first keeps the poll out of
        // the queue behind the sixteen loads below.
        mbar_wait_n(&S.g_full[sl], n_gfull[sl]++, failed);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // The chunk's last gradient product has completed: its rows make room for those of the chunk after
        // the next, so that the issuer always has the next chunk's rows when a slot falls free.
        if (last) {
          if (c + 2 < nch) load_x_tile(sm + kOffX + (c & 1) * kB * kCh * 2, idx, c + 2);
          asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (u + 1 < NU) {   // the master rows of the next unit: on their way during this unit's work
          const float* src = work + oW0 + w0_block((u + 1) / UPC, unit_hh(u + 1), half) + r * 4;
#pragma unroll
          for (int k = 0; k < 16; ++k) wn[k] = *reinterpret_cast<const float4*>(src + k * 512);
        }
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {
          uint32_t v[32];
          tmem_ld32(tq + kColG + 128 * sl + 64 * half + 32 * hb, v);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            float4& x = w[8 * hb + k];
            x.x = fmaf(-eta, fmaf(lambda, x.x, __uint_as_float(v[4 * k])), x.x);
            x.y = fmaf(-eta, fmaf(lambda, x.y, __uint_as_float(v[4 * k + 1])), x.y);
            x.z = fmaf(-eta, fmaf(lambda, x.z, __uint_as_float(v[4 * k + 2])), x.z);
            x.w = fmaf(-eta, fmaf(lambda, x.w, __uint_as_float(v[4 * k + 3])), x.w);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&S.g_free[sl]);       // the slot may take the gradient of unit u + 2
        // Shared-memory work first, the master's stores last: the proxy fence below would otherwise
        // wait for sixteen global stores per thread on every unit.
        if (fuse && u >= 1) mbar_wait_n(&S.wn_free, n_wnfree++, failed);   // the forward product of unit u - 1 has read the unit tile
        if (first && more) {
          // rows of the next chunk for the forward product: their buffer was last read by the forward
          // products of chunk c - 1, the last of which was waited for just now
          if (fuse) load_x_tile(sm + kOffX + (2 + ((c + 1) & 1)) * kB * kCh * 2, idxn, c + 1);
          asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (fuse) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            uint4 o;
            o.x = pack_bf16(w[2 * k].x, w[2 * k].y); o.y = pack_bf16(w[2 * k].z, w[2 * k].w);
            o.z = pack_bf16(w[2 * k + 1].x, w[2 * k + 1].y); o.w = pack_bf16(w[2 * k + 1].z, w[2 * k + 1].w);
            *reinterpret_cast<uint4*>(sm + kOffWn + tile_off(r, 64 * half + 8 * k, 128)) = o;
          }
        }
        // What must have landed before the arrivals below: the gradient rows of chunk c + 2 (for the
        // issuer), the forward rows of chunk c (read by the product that takes this unit tile), and
        // for a single CTA those of chunk c + 1, whose first unit has no wait of its own.  In a pair the
        // forward rows of chunk c + 1, the group committed last, may stay in flight until the next unit.
        const bool rows_due = last && c + 2 < nch;
        if (last) {
          if (NR == 2 && more) asm volatile("cp.async.wait_group 1;" ::: "memory");
          else asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        if (fuse || rows_due) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            if (fuse) mbar_arrive(&S.wn_ready);
            if (rows_due) mbar_arrive(&S.x_ready[c & 1]);
          }
        }
#pragma unroll
        for (int k = 0; k < 16; ++k) *reinterpret_cast<float4*>(dst + k * 512) = w[k];
      }
      if (fuse) mbar_wait_n(&S.wn_free, n_wnfree++, failed);   // the last unit's forward product
    } else {
      // ---- the issuing warp ----
      const uint32_t idg = idesc_bf16(128, 128, 1, 0), idf = idesc_bf16(128, kB, 1, 0);
      auto issue_fwd = [&](int u) {
        const int c = u / UPC, hh = unit_hh(u);
        mbar_wait_n(&S.wn_ready, n_wnready++, failed);
        if (lane == 0 && !failed) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t xs = sX + (2 + (c & 1)) * kB * kCh * 2;
          for (int ks = 0; ks < kCh / 16; ++ks)
            umma_bf16(tmem + kColZ0 + (NR == 1 ? 64 * hh : 0), view_mn(sWn, 128, 0, ks * 16), view_k(xs, kCh, 0, ks * 16), idf, (c > 0 || ks > 0) ? 1u : 0u);
        }
        if (lane == 0) umma_commit(&S.wn_free);
        __syncwarp();
      };
      for (int u = 0; u < NU; ++u) {
        const int c = u / UPC, hh = unit_hh(u), sl = u & 1;
        if (u % UPC == 0) { mbar_wait_n(&S.x_ready[c & 1], n_xready[c & 1]++, failed); }
        if (u >= 2) mbar_wait_n(&S.g_free[sl], n_gfree[sl]++, failed);
        if (lane == 0 && !failed) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t xs = sX + (c & 1) * kB * kCh * 2;
          for (int ks = 0; ks < kB / 16; ++ks)
            umma_bf16(tmem + kColG + 128 * sl, view_mn(xs, kCh, 0, ks * 16), view_k(sdZ0, kB, NR == 1 ? 128 * hh : 0, ks * 16), idg, ks > 0 ? 1u : 0u);
        }
        if (lane == 0) umma_commit(&S.g_full[sl]);
        __syncwarp();
        if (fuse && u >= 1) issue_fwd(u - 1);
      }
      if (fuse) issue_fwd(NU - 1);
      // the epilogue's last two slot releases complete a phase nobody waits for: keep the count in step
      if (NU >= 2) { n_gfree[0]++; n_gfree[1]++; }
      else if (NU == 1) n_gfree[0]++;
    }
    __syncthreads();
    // the other side's counters: both sides saw the same number of completions
    if (ewarp) {
      n_wnready += fuse ? (uint32_t)NU : 0u;
      n_xready[0] += (uint32_t)((nch + 1) / 2); n_xready[1] += (uint32_t)(nch / 2);
      n_gfree[0] += (uint32_t)((NU + 1) / 2); n_gfree[1] += (uint32_t)(NU / 2);
    } else {
      n_gfull[0] += (uint32_t)((NU + 1) / 2); n_gfull[1] += (uint32_t)(NU / 2);
      n_wnfree += fuse ? (uint32_t)NU : 0u;
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }

  // ---- event trigger: publish (c, U_i, i); of a pair, each CTA the blocks it owns ----
  __syncthreads();
  {
    const float inv_eta = 1.f / eta;
    float* wend = p.r.w_end ? p.r.w_end + (size_t)t.u_row * p.r.stride : nullptr;
    // U = (w_start - w_end) / eta, piece by piece, in the natural order and eight pieces per thread and trip as at the start
    constexpr int kTrip = 8;
    auto finish_range = [&](size_t total, size_t o_layer, auto where) {
      for (size_t base = tid; base < total; base += (size_t)kTrip * kSThreads) {
        float4 w[kTrip], a[kTrip];
        size_t jj[kTrip], dd[kTrip];
#pragma unroll
        for (int q = 0; q < kTrip; ++q) {
          const size_t e4 = base + (size_t)q * kSThreads;
          where(e4 < total ? e4 : 0, jj[q], dd[q]);
          w[q] = *reinterpret_cast<const float4*>(work + o_layer + 4 * dd[q]);
          a[q] = *reinterpret_cast<const float4*>(Urow + jj[q]);
        }
#pragma unroll
        for (int q = 0; q < kTrip; ++q)
          if (base + (size_t)q * kSThreads < total) {
            *reinterpret_cast<float4*>(Urow + jj[q]) = make_float4((a[q].x - w[q].x) * inv_eta, (a[q].y - w[q].y) * inv_eta,
                                                                     (a[q].z - w[q].z) * inv_eta, (a[q].w - w[q].w) * inv_eta);
            if (wend) *reinterpret_cast<float4*>(wend + jj[q]) = w[q];
          }
      }
    };
    constexpr int kColQ = kH0 / 4 / NR;
    finish_range((size_t)D0 * kColQ, oW0, [&](size_t e4, size_t& j, size_t& d4) {
      const int i = (int)(e4 / kColQ), q = (int)(e4 % kColQ) + (NR == 2 ? rank * kColQ : 0);
      const int c = i >> 7, r = i & 127, hh = q >> 5, half = (q >> 4) & 1, k = q & 15;
      d4 = ((size_t)((c * 2 + hh) * 2 + half) << 11) + ((size_t)k << 7) + r;
      j = oW0 + (size_t)i * kH0 + 4 * q;
    });
    finish_range((size_t)kH0 * kH1 / 4 / NR, oW1, [&](size_t e4, size_t& j, size_t& d4) {
      const int i = (int)(e4 / (kH1 / 4)) + (NR == 2 ? rank * 128 : 0), q = (int)(e4 % (kH1 / 4));
      const int tl = i >> 7, r = i & 127, g32 = q >> 3, k = q & 7;
      d4 = ((size_t)(tl * 4 + g32) << 10) + ((size_t)k << 7) + r;
      j = oW1 + (size_t)i * kH1 + 4 * q;
    });
    // the narrow parameters: identical in both CTAs of a pair except the first bias, of which each holds its half
    for (int j = tid; j < kH0 + kH1 + kH1 * C + C; j += kSThreads) {
      const size_t g = j < kH0 ? ob0 + j : (j < kH0 + kH1 ? ob1 + (j - kH0) : oW2 + (j - kH0 - kH1));
      if (NR == 2 && (j < kH0 ? (j >> 7) != rank : rank != 0)) continue;
      float u, w;
      if (g < oW1) { u = S.Ub0[g - ob0]; w = S.b0[g - ob0]; }
      else if (g < oW2) { u = S.Ub1[g - ob1]; w = S.b1[g - ob1]; }
      else if (g < ob2) { u = S.UW2[g - oW2]; w = S.W2[g - oW2]; }
      else { u = S.Ub2[g - ob2]; w = S.b2[g - ob2]; }
      Urow[g] = u;
      if (wend) wend[g] = w;
    }
  }
  if (failed) atomicOr(&S.failed, 1u);
  __syncthreads();
  if (tid == 0) {
    if (S.failed && p.r.status) atomicOr(p.r.status, 1u);
    if (rank == 0) {
      TriggerRec rec;
      rec.client = t.client; rec.round = t.round; rec.samples_done = t.steps * (uint32_t)kB; rec.flags = 1;
      p.r.trig[t.seq] = rec;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (NR == 2) cluster_sync(); else __syncthreads();   // pair: the peer has stopped writing into this CTA's shared memory
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

bool mlp_stream_eligible(const MlpShape& s) {
  return s.precision == 1 && s.n_layers == 3 && s.dims[1] == (uint32_t)kH0 && s.dims[2] == (uint32_t)kH1 &&
         s.dims[3] <= (uint32_t)kMaxC && s.dims[0] >= 256 && s.dims[0] % (2 * kCh) == 0 && s.batch == (uint32_t)kB;
}

cudaError_t launch_mlp_stream_rounds(const MlpLaunch& p, cudaStream_t s) {
  if (p.r.n_tasks == 0) return cudaSuccess;
  int sms = 0;   // asked of the current device at every launch: cheap, and right on any device of the process
  {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  // two SMs per round-task while the launch leaves that many free; a fuller launch runs one CTA per round-task
  const bool pair = 2 * (int)p.r.n_tasks <= sms;
  cudaError_t e = cudaFuncSetAttribute(pair ? mlp_stream_kernel<2> : mlp_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (e != cudaSuccess) return e;
  if (!pair) {
    mlp_stream_kernel<1><<<p.r.n_tasks, kSThreads, kSmemBytes, s>>>(p);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.r.n_tasks * 2, 1, 1);
  cfg.blockDim = dim3(kSThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, mlp_stream_kernel<2>, p);
}

}  // namespace aet
