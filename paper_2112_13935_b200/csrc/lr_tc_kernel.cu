// Local-SGD round of one client for softmax regression 784 -> 10, batch 1, lambda = 0, for
// launches with more round-tasks than SMs: the update sum lives in tensor memory and is
// accumulated by the tensor cores.
//
// Algorithm 3, MainComputeNode, inner loop ("g = grad f(w_c, xi); w_c -= eta_i g; U_i += g"),
// taken kM = 8 steps at a time exactly as lr_block_kernel does: with W the model at the start of
// a block, delta_s = softmax(z_s) - onehot(y_s) and G[s][t] = x_s . x_t + 1,
//     z_t = W x_t + b - eta * sum_{s<t} delta_s G[s][t],      W = W_start - eta * U.
// What differs is where the work runs:
//   P1  eight warps; warp = (quarter q of tensor memory's 128 lanes, class half ch).  Thread
//       (q, l, ch) owns the "pixels" 128 j + 32 q + l, j = 0..6 (pixel 784 is the bias, an always-1
//       input) and classes 5 ch .. 5 ch + 4: it reads its entries of U from tensor memory
//       (tcgen05.ld), forms W = W_start - eta U, adds its share of Z0 = W X, and writes its pixels
//       of the block's eight rows into the tensor cores' operand tiles, split into a tf32 head and
//       an fp32 remainder (hi written by the ch = 0 warps, lo by the ch = 1 warps);
//   R   one warp (rotating) takes the eight dependent softmax steps - or, when the coupling
//       eta * G is small, sweeps all eight at once until the logits stop moving (see below) -
//       while three warps compute the Gram matrix of the next block and one issues the row
//       copies of the block after it;
//   U   U^T[pixel, class] += X^T[pixel, sample] . delta[sample, class] is one tcgen05.mma
//       (kind::tf32, M = 128 pixels, N = 16, K = 8 samples) per 128-pixel tile and term:
//       hi.hi + lo.hi + hi.lo, fp32 accumulation in tensor memory (7 x 16 columns).  The product
//       of the two remainders (2^-22 relative) is dropped.
// The update sum never passes through registers between blocks, the FMA work per sample drops
// from 2.25 to 1.25 per parameter, and the softmax chain of one CTA overlaps the FMA phase of the
// CTA sharing the SM.  Operand tiles use the K-major no-swizzle core-matrix layout (8 rows x 16
// bytes; LBO = stride between core matrices along K, SBO = along M/N).  Every mbarrier wait is
// bounded; a wait that runs out flags `status`, and the CTA still frees its tensor memory.
//
// Fixed-point form of R.  The eight corrected logits solve z = Z0 + L delta(z) with L strictly
// lower triangular (L[t][s] = -eta G[s][t] for s < t), which the step-by-step walk solves by
// substitution.  Sweeping z <- Z0 + L delta(z) over all samples at once reaches the same
// solution: after i sweeps the first i samples are exact (so eight sweeps always suffice), and
// the error shrinks by rho = max_t sum_s |L[t][s]| / 2 per sweep (the softmax has Lipschitz
// constant 1/2 in the maximum norm).  The sweeps stop as soon as rho / (1 - rho) times the last
// change of the logits is below 2e-7; one more softmax then gives delta to fp32 round-off.  With
// rho > 1/4 the walk is taken step by step.
#include <cuda_runtime.h>

#include "aet_kernels.h"
#include "aet_rng.h"
#include "lr_common.cuh"

namespace aet {
namespace {

using namespace lr;

constexpr int kTcWarps = 8, kTcThreads = kTcWarps * 32;
constexpr int kTiles = 7;          // 128-row tiles of the 785 inputs (784 pixels + the bias input)
constexpr int kRing = 2;           // blocks of rows in shared memory
constexpr int kLabelRing = 4;      // blocks of labels: the labels of block k + 2 are written while R still reads those of block k
constexpr int kGramRanks = 3;      // warps sharing the Gram matrix of a block
constexpr uint32_t kTmemCols = 128;
constexpr float kSweepTol = 2e-7f;

struct __align__(128) TcSmem {
  float rows[kRing][kM][kD];       // the sampled rows as they arrive
  float A[2][kTiles][2][128][4];   // operand tiles [hi | lo][tile][k group][row][4 samples]; the first kStageFloats
                                   // floats double as the staging area of a model row before and after the round
  float B[2][2][16][4];            // delta [hi | lo][k group][column n][4 samples]; class c sits in column c (c < 5) or c + 3
  float partZ[4][kM * kC];         // Z0 partial sums per quarter, index t * 10 + c
  float partG[2][kGramRanks][32];  // Gram pair partial sums, double-buffered by block parity
  float consts[8];                 // [0] = 1 (the bias input), [4] = 0 (rows no pixel maps to)
  int ys[kLabelRing][kM];
  uint64_t full[kRing];
  uint64_t staged;
  uint64_t delta_ready;            // R has written the block's delta operand
  uint64_t mma_done;               // the seven tiles' products of a block have completed
  uint32_t tmem_base;
};
static_assert(sizeof(float) * 2 * kTiles * 2 * 128 * 4 >= sizeof(float) * kStageFloats, "staging area fits the operand tiles");
static_assert(sizeof(TcSmem) <= 114 * 1024, "two CTAs per SM");

__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {   // K-major, no swizzle
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  return d;
}
// Instruction descriptor: tf32 x tf32 -> fp32, both operands K-major, M = 128, N = 16.
constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(kIdesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld8_issue(uint32_t taddr, uint32_t (&v)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Nearest tf32 (10 stored mantissa bits, low 13 bits of the word zero) of a finite fp32, as fp32:
// exactly representable in the tensor cores' input format whatever they do with the low bits.
__device__ __forceinline__ float tf32_head(float v) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
  return __uint_as_float(r);
}

template <bool kSweep>
__global__ void __launch_bounds__(kTcThreads, 2) lr_tc_kernel(RoundLaunch p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TcSmem& sm = *reinterpret_cast<TcSmem*>(smem_raw);
  float* stage = &sm.A[0][0][0][0][0];

  const TaskDesc t = p.tasks[p.task_begin + blockIdx.x];
  if (!debug_task_ok(p, t)) return;   // debug checks only: rows and slots in range, else flag and skip
  if (t.n_samples == 0) {   // this grid may run under the tail of the aggregation before it: wait before writing
    asm volatile("griddepcontrol.wait;" ::: "memory");
    publish_empty_round(p, t, kParams);
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q = warp & 3, ch = warp >> 2;
  const int row = 32 * q + lane;                        // this thread's row of every 128-row tile
  // tile 6 holds pixels 768..783 in rows 0..15 and the bias input in row 16
  const bool pix6 = row < 16, bias6 = row == 16;

  const ClientData cd = p.clients[t.client];
  const uint64_t key = p.sample_keys[t.client];
  const float* xrows = reinterpret_cast<const float*>(cd.x);
  const uint32_t n = t.n_samples;
  const uint32_t nblk = (n + kM - 1) / kM;
  const float neta = -t.eta;

  if (threadIdx.x == 0) {
#pragma unroll
    for (int s = 0; s < kRing; ++s) mbar_init(&sm.full[s], 1);
    mbar_init(&sm.staged, 1);
    mbar_init(&sm.delta_ready, 1);
    mbar_init(&sm.mma_done, kTiles);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 8) sm.consts[threadIdx.x] = threadIdx.x == 0 ? 1.f : 0.f;
  if (threadIdx.x < 2 * 2 * 16 * 4) (&sm.B[0][0][0][0])[threadIdx.x] = 0.f;   // the six unused columns stay zero
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&sm.tmem_base)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tmem_mine = tmem + ((uint32_t)(32 * q) << 16) + 8u * ch;   // this warp's lanes, this class half's columns

  // Producer step: the rows and labels of block kb into ring slot kb % kRing.
  auto produce = [&](uint32_t kb) {
    const int sb = kb % kRing;
    const uint32_t nvb = min((uint32_t)kM, n - kb * kM);
    // a short last block: the rows nobody copies are zeroed, so that they add nothing anywhere; the
    // warp barrier puts these stores ahead of lane 0's arrival, which is what the readers wait for
    for (uint32_t r = nvb; r < (uint32_t)kM; ++r)
      for (int i = lane; i < kD; i += 32) sm.rows[sb][r][i] = 0.f;
    __syncwarp();
    if (lane == 0) mbar_expect_tx(&sm.full[sb], nvb * kRowBytes);
    __syncwarp();
    if ((uint32_t)lane < nvb) {
      const uint32_t idx = sample_index(draw(key, t.sample_ctr0 + kb * kM + lane), cd.n);
      bulk_load_row(sm.rows[sb][lane], xrows + (size_t)idx * kD, &sm.full[sb]);
      sm.ys[kb % kLabelRing][lane] = __ldg(cd.y + idx);
    }
  };

  // ---- start model: server snapshot minus own update sums still in flight ----
  // ws[j][c] = W_start[128 j + row][5 ch + c]; row 16 of tile 6 holds the biases.
  float ws[kTiles][kCh];
  bool ok = true;
  {
#pragma unroll
    for (int j = 0; j < kTiles; ++j)
#pragma unroll
      for (int c = 0; c < kCh; ++c) ws[j][c] = 0.f;
    // Everything above reads only what earlier, finished grids and the host wrote.  The snapshot is
    // written by the aggregation kernel launched just before this grid, which may still be running
    // when this grid was launched with programmatic stream serialisation.
    if (warp == 0) produce(0);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // The snapshot and the first update sum in flight (nine round-tasks in ten have exactly one) come in
    // side by side: the snapshot into the staging area, the sum behind it in what is left of the operand
    // tiles, its last 5.6 KB in the second block of rows, whose copies are issued only afterwards.
    constexpr int kHeadFloats = 2 * kTiles * 2 * 128 * 4 - kStageFloats, kTailFloats = kStageFloats - kHeadFloats;
    static_assert(kHeadFloats > 0 && kHeadFloats % 4 == 0 && kTailFloats % 4 == 0 && kTailFloats <= kM * kD, "second staging area");
    const float* head2 = stage + kStageFloats;
    const float* tail2 = &sm.rows[1][0][0];
    const uint32_t nfl = t.inflight_cnt;
    float scale2 = 0.f;
    if (nfl) scale2 = -p.inflight[t.inflight_off].eta;
    if (threadIdx.x == 0) {
      mbar_expect_tx(&sm.staged, (nfl ? 2u : 1u) * kStageFloats * sizeof(float));
      bulk_load(stage, p.snaps + (size_t)t.snap_slot * p.stride, kStageFloats * sizeof(float), &sm.staged);
      if (nfl) {
        const float* src = p.U + (size_t)p.inflight[t.inflight_off].row * p.stride;
        bulk_load(const_cast<float*>(head2), src, kHeadFloats * sizeof(float), &sm.staged);
        bulk_load(const_cast<float*>(tail2), src + kHeadFloats, kTailFloats * sizeof(float), &sm.staged);
      }
    }
    ok = mbar_wait(&sm.staged, 0) && ok;
#pragma unroll
    for (int j = 0; j < kTiles; ++j) {
      const bool live = j < kTiles - 1 || pix6 || bias6;
#pragma unroll
      for (int c = 0; c < kCh; ++c) {
        const int e = (128 * j + row) * kC + kCh * ch + c;
        float v = live ? stage[e] : 0.f;
        if (nfl && live) v = fmaf(scale2, e < kHeadFloats ? head2[e] : tail2[e - kHeadFloats], v);
        ws[j][c] = v;
      }
    }
    for (uint32_t f = 1; f < nfl; ++f) {   // further sums in flight, one after the other
      const InflightRef ref = p.inflight[t.inflight_off + f];
      __syncthreads();   // everybody has taken the previous row out of the staging area
      if (threadIdx.x == 0) {
        mbar_expect_tx(&sm.staged, kStageFloats * sizeof(float));
        bulk_load(stage, p.U + (size_t)ref.row * p.stride, kStageFloats * sizeof(float), &sm.staged);
      }
      ok = mbar_wait(&sm.staged, f & 1) && ok;
#pragma unroll
      for (int j = 0; j < kTiles; ++j) {
        const bool live = j < kTiles - 1 || pix6 || bias6;
#pragma unroll
        for (int c = 0; c < kCh; ++c) {
          const float v = live ? stage[(128 * j + row) * kC + kCh * ch + c] : 0.f;
          ws[j][c] = fmaf(-ref.eta, v, ws[j][c]);
        }
      }
    }
    __syncthreads();   // the staging areas become the operand tiles and the second block of rows
    if (warp == 0 && nblk > 1) produce(1);
  }

  // Where this thread reads its input of sample s for tiles 0..5 and for tile 6.
  const float* x05 = &sm.rows[0][0][row];
  const float* x6 = pix6 ? &sm.rows[0][0][768 + row] : (bias6 ? &sm.consts[0] : &sm.consts[4]);
  const int rs6 = pix6 ? kD : 0;

  static_assert(BflyDims<kM * kCh>::n5 == 2 && BflyDims<kPairs>::n5 == 1, "butterfly widths");
  int zidx[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int v = bfly_index5<kM * kCh>(lane, i);       // v = s * 5 + c
    zidx[i] = v < 0 ? -1 : (v / kCh) * kC + ch * kCh + (v % kCh);
  }
  const int gidx = bfly_index5<kPairs>(lane, 0);

  // Gram pairs of block kb over this warp's share of the pixels (rank r of kGramRanks).
  auto gram_partial = [&](uint32_t kb, int r) {
    const float* rb = &sm.rows[kb % kRing][0][0];
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
    if (gidx >= 0) sm.partG[kb & 1][r][gidx] = o[0];
  };

  bool timed_out = false;
  uint32_t timeout_at = 0;

  if (warp >= 1 && warp <= kGramRanks) {   // Gram matrix of block 0 (warp 0 runs R for block 0)
    ok = mbar_wait(&sm.full[0], 0) && ok;
    gram_partial(0, warp - 1);
  }

  for (uint32_t k = 0; k < nblk; ++k) {
    const int slot = k % kRing;
    const uint32_t nv = min((uint32_t)kM, n - k * kM);
    ok = mbar_wait(&sm.full[slot], (k / kRing) & 1) && ok;
    if (k) {   // the tensor cores have added block k-1 to U and are done with the operand tiles
      ok = mbar_wait(&sm.mma_done, (k - 1) & 1) && ok;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }

    // ---- P1: W = W_start - eta U; this thread's share of Z0 = W X; operand tiles of the block ----
    {
      float acc[kM][kCh];
#pragma unroll
      for (int s = 0; s < kM; ++s)
#pragma unroll
        for (int c = 0; c < kCh; ++c) acc[s][c] = 0.f;
      const float* xs05 = x05 + (size_t)slot * kM * kD;
      const float* xs6 = x6 + (size_t)slot * kM * rs6;
      uint32_t u[8], un[8];
      if (k) tmem_ld8_issue(tmem_mine, u);
#pragma unroll
      for (int j = 0; j < kTiles; ++j) {
        float W[kCh];
        if (k) {
          tmem_ld_wait();
          if (j + 1 < kTiles) tmem_ld8_issue(tmem_mine + 16u * (j + 1), un);
#pragma unroll
          for (int c = 0; c < kCh; ++c) W[c] = fmaf(neta, __uint_as_float(u[c]), ws[j][c]);
        } else {
#pragma unroll
          for (int c = 0; c < kCh; ++c) W[c] = ws[j][c];
        }
        const float* xp = j < kTiles - 1 ? xs05 + 128 * j : xs6;
        const int rs = j < kTiles - 1 ? kD : rs6;
        float x[kM];
#pragma unroll
        for (int s = 0; s < kM; ++s) x[s] = xp[s * rs];   // rows of a short last block were zeroed by the producer
#pragma unroll
        for (int s = 0; s < kM; ++s)
#pragma unroll
          for (int c = 0; c < kCh; ++c) acc[s][c] = fmaf(x[s], W[c], acc[s][c]);
        float o8[kM];
        if (ch == 0) {   // warp-uniform: the heads
#pragma unroll
          for (int s = 0; s < kM; ++s) o8[s] = tf32_head(x[s]);
        } else {         // the remainders
#pragma unroll
          for (int s = 0; s < kM; ++s) o8[s] = x[s] - tf32_head(x[s]);
        }
        *reinterpret_cast<float4*>(&sm.A[ch][j][0][row][0]) = make_float4(o8[0], o8[1], o8[2], o8[3]);
        *reinterpret_cast<float4*>(&sm.A[ch][j][1][row][0]) = make_float4(o8[4], o8[5], o8[6], o8[7]);
        if (k && j + 1 < kTiles) {
#pragma unroll
          for (int c = 0; c < 8; ++c) u[c] = un[c];
        }
      }
      float v[kM * kCh];
#pragma unroll
      for (int s = 0; s < kM; ++s)
#pragma unroll
        for (int c = 0; c < kCh; ++c) v[s * kCh + c] = acc[s][c];
      float o[2];
      bfly_reduce5<kM * kCh>(v, o, lane);
#pragma unroll
      for (int i = 0; i < 2; ++i)
        if (zidx[i] >= 0) sm.partZ[q][zidx[i]] = o[i];
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor cores read the tiles written above
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    // barrier A: partial sums and operand tiles visible, rows of block k no longer read by anyone; it
    // also carries the verdict of the bounded waits so that all threads leave together
    if (__syncthreads_or(!ok)) { timed_out = true; timeout_at = k; break; }

    const int rwarp = (int)(k & (kTcWarps - 1));
    const int rel = (warp - rwarp) & (kTcWarps - 1);
    if (rel == 0) {
      // ---- R: the block's kM dependent softmax steps.  Four lanes share a sample: lane 4 j + g owns
      // classes g, g + 4 and (g < 2) g + 8 of sample j, so that a sweep costs 21 shuffles instead of 70.
      const int j = lane >> 2, g = lane & 3;
      constexpr int kOwn = 3;
      constexpr float kNoClass = -1e30f;   // stands in for the third class of g >= 2: exp gives 0, nothing moves
      float z[kOwn];
#pragma unroll
      for (int i = 0; i < kOwn; ++i) {
        const int c = g + 4 * i;
        const int at = j * kC + (c < kC ? c : 0);
        const float v = (sm.partZ[0][at] + sm.partZ[1][at]) + (sm.partZ[2][at] + sm.partZ[3][at]);
        z[i] = c < kC ? v : kNoClass;
      }
      const float* g0 = sm.partG[k & 1][0];
      const float* g1 = sm.partG[k & 1][1];
      const float* g2 = sm.partG[k & 1][2];
      const int gbase = j * (j - 1) / 2;
      // -eta * G[s][j] for s < j, 0 for the others (a finished sample takes no correction)
      auto corr = [&](int s) -> float {
        const int idx = s < j ? gbase + s : 0;
        const float gsum = (1.f + g0[idx]) + (g1[idx] + g2[idx]);   // 1 = the bias input
        return s < j && (uint32_t)j < nv ? gsum * neta : 0.f;
      };
      const int y = sm.ys[k % kLabelRing][j];
      float oh[kOwn];
#pragma unroll
      for (int i = 0; i < kOwn; ++i) oh[i] = g + 4 * i == y ? -1.f : 0.f;
      auto softmax_delta = [&](const float (&zz)[kOwn], float (&d)[kOwn]) {
        float m = fmaxf(fmaxf(zz[0], zz[1]), zz[2]);
        m = fmaxf(m, shx(m, 1));
        m = fmaxf(m, shx(m, 2));
        const float nms = -m * kLog2e;
        float e[kOwn];
#pragma unroll
        for (int i = 0; i < kOwn; ++i) e[i] = ex2(fmaf(zz[i], kLog2e, nms));
        float sum = (e[0] + e[1]) + e[2];
        sum += shx(sum, 1);
        sum += shx(sum, 2);
        const float inv = rcp(sum);
#pragma unroll
        for (int i = 0; i < kOwn; ++i) d[i] = fmaf(e[i], inv, oh[i]);
      };
      float dk[kOwn];   // delta of this lane's own sample and classes
#pragma unroll
      for (int i = 0; i < kOwn; ++i) dk[i] = 0.f;

      bool swept = false;
      if (kSweep) {
        // all couplings of this lane's sample at once: L[j][s] for s < j
        float Lr[kM - 1];
        float rowsum = 0.f;
#pragma unroll
        for (int s = 0; s < kM - 1; ++s) { Lr[s] = corr(s); rowsum += fabsf(Lr[s]); }
        float rho = rowsum;
        rho = fmaxf(rho, shx(rho, 16)); rho = fmaxf(rho, shx(rho, 8)); rho = fmaxf(rho, shx(rho, 4));
        rho *= 0.5f;
        if (rho <= 0.25f) {
          swept = true;
          const float gain = rho / (1.f - rho);
          float z0[kOwn];
#pragma unroll
          for (int i = 0; i < kOwn; ++i) z0[i] = z[i];
          // at most nv sweeps are ever needed: sweep i makes the first i samples exact
          for (uint32_t sweep = 0; sweep < nv; ++sweep) {
            float d[kOwn];
            softmax_delta(z, d);
            float zn[kOwn];
#pragma unroll
            for (int i = 0; i < kOwn; ++i) zn[i] = z0[i];
#pragma unroll
            for (int s = 0; s < kM - 1; ++s)
#pragma unroll
              for (int i = 0; i < kOwn; ++i) zn[i] = fmaf(__shfl_sync(0xffffffffu, d[i], 4 * s + g), Lr[s], zn[i]);
            float change = 0.f;
#pragma unroll
            for (int i = 0; i < kOwn; ++i) { change = fmaxf(change, fabsf(zn[i] - z[i])); z[i] = zn[i]; }
            if (!__any_sync(0xffffffffu, change * gain > kSweepTol)) break;
          }
          softmax_delta(z, dk);
        }
      }
      if (!swept) {
        float gs = corr(0);
        // The loop stays rolled: the whole per-block body has to fit the instruction cache.
#pragma unroll 1
        for (int s = 0; s < (int)nv; ++s) {
          const float gnext = corr(s + 1);
          float d[kOwn];
          softmax_delta(z, d);
          const bool mine = j == s;
#pragma unroll
          for (int i = 0; i < kOwn; ++i) {
            dk[i] = mine ? d[i] : dk[i];
            z[i] = fmaf(__shfl_sync(0xffffffffu, d[i], 4 * s + g), gs, z[i]);
          }
          gs = gnext;
        }
      }
      // delta as the tensor cores' second operand: tf32 head and remainder, zero for missing samples
      {
        const bool live = (uint32_t)j < nv;
#pragma unroll
        for (int i = 0; i < kOwn; ++i) {
          const int c = g + 4 * i;
          if (c < kC) {
            const float d = live ? dk[i] : 0.f;
            const float hi = tf32_head(d);
            const int col = c < kCh ? c : c + 3;
            sm.B[0][j >> 2][col][j & 3] = hi;
            sm.B[1][j >> 2][col][j & 3] = d - hi;
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&sm.delta_ready)) : "memory");
    } else if (rel <= kGramRanks) {
      if (k + 1 < nblk) {
        ok = mbar_wait(&sm.full[(k + 1) % kRing], ((k + 1) / kRing) & 1) && ok;
        gram_partial(k + 1, rel - 1);
      }
    } else if (rel == kGramRanks + 1) {
      // block k+2 takes the slot of block k: free since barrier A
      if (k + 2 < nblk) produce(k + 2);
    }
    if (rel != 0) {
      // ---- U: U^T += X^T delta on the tensor cores, hi.hi + lo.hi + hi.lo.  Each of the seven warps
      // other than R issues the three products of one 128-pixel tile (an instruction keeps its
      // issuing thread for some 80 cycles, whatever its size) and commits them to mma_done.
      ok = mbar_wait(&sm.delta_ready, k & 1) && ok;
      if (lane == 0 && ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int jt = rel - 1;
        const uint64_t bhi = umma_desc(smem_addr(&sm.B[0][0][0][0]), 256, 128);
        const uint64_t blo = umma_desc(smem_addr(&sm.B[1][0][0][0]), 256, 128);
        const uint64_t ahi = umma_desc(smem_addr(&sm.A[0][jt][0][0][0]), 2048, 128);
        const uint64_t alo = umma_desc(smem_addr(&sm.A[1][jt][0][0][0]), 2048, 128);
        const uint32_t d = tmem + 16u * jt;
        umma_tf32(d, ahi, bhi, k ? 1u : 0u);
        umma_tf32(d, alo, bhi, 1u);
        umma_tf32(d, ahi, blo, 1u);
        umma_commit(&sm.mma_done);
      }
      __syncwarp();
    }
  }

  if (!timed_out) {
    // the last block's product; the barrier carries the verdict of the waits since barrier A
    ok = mbar_wait(&sm.mma_done, (nblk - 1) & 1) && ok;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (__syncthreads_or(!ok)) { timed_out = true; timeout_at = nblk; }
  }

  if (timed_out) {
    // A copy or a product never completed.  Flag it and give the copies still in flight a bounded
    // chance to land (their target is this CTA's shared memory).
    if (threadIdx.x == 0) {
      if (p.status) atomicOr(p.status, 1u);
      for (uint32_t j = timeout_at; j < nblk && j < timeout_at + 2; ++j) mbar_wait(&sm.full[j % kRing], (j / kRing) & 1);
      mbar_wait(&sm.staged, (t.inflight_cnt > 1 ? t.inflight_cnt - 1 : 0) & 1);   // the last rows staged at the start
    }
  } else {
    // The aggregation kernel behind this grid in the stream may become resident from here on (it
    // touches nothing until this grid has finished and its writes are visible).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // ---- event trigger: h reached s_{i,c}; publish U_i (and the end model W_start - eta U) ----
    float Uv[kTiles][kCh];
    {
      uint32_t u[8];
#pragma unroll
      for (int j = 0; j < kTiles; ++j) {
        tmem_ld8_issue(tmem_mine + 16u * j, u);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < kCh; ++c) Uv[j][c] = __uint_as_float(u[c]);
      }
    }
    for (int pass = 0; pass < (p.w_end ? 2 : 1); ++pass) {
      float* dst = (pass == 0 ? p.U : p.w_end) + (size_t)t.u_row * p.stride;
      if (pass) __syncthreads();   // the previous row has left the staging area
      if (threadIdx.x < kStageFloats - kParams) stage[kParams + threadIdx.x] = 0.f;   // the row's padding
#pragma unroll
      for (int j = 0; j < kTiles; ++j) {
        const bool live = j < kTiles - 1 || pix6 || bias6;
        if (live) {
#pragma unroll
          for (int c = 0; c < kCh; ++c)
            stage[(128 * j + row) * kC + kCh * ch + c] = pass == 0 ? Uv[j][c] : fmaf(neta, Uv[j][c], ws[j][c]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the bulk copy reads what the threads wrote
      __syncthreads();
      if (threadIdx.x == 0) bulk_store_and_wait(dst, stage, kStageFloats * sizeof(float));
    }
    if (threadIdx.x == 0) {
      TriggerRec rec;
      rec.client = t.client; rec.round = t.round; rec.samples_done = n; rec.flags = 1;
      p.trig[t.seq] = rec;
    }
  }

  // tensor memory goes back on every path
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

bool lr_tc_eligible(const RoundLaunch& p) { return p.l2 == 0.f && p.stride == (size_t)lr::kStageFloats; }

cudaError_t launch_lr_tc_rounds(const RoundLaunch& p, cudaStream_t s) {
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool known = dev >= 0 && dev < 64;
  if (!known || !opted_in[dev]) {
    e = cudaFuncSetAttribute(lr_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(lr_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
    if (e != cudaSuccess) return e;
    if (known) opted_in[dev] = true;
  }
  // Programmatic stream serialisation, as for lr_block_kernel: the grid may start under the tail of
  // the aggregation kernel ahead of it and waits (griddepcontrol.wait) before reading its output.
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.n_tasks, 1, 1);
  cfg.blockDim = dim3(kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = sizeof(TcSmem);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return p.step_by_step ? cudaLaunchKernelEx(&cfg, lr_tc_kernel<false>, p) : cudaLaunchKernelEx(&cfg, lr_tc_kernel<true>, p);
}

}  // namespace aet
