// Launch interfaces of the device kernels (plain structs, no library types).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "aet_schedule.h"

namespace aet {

// Device view of one client's local data set D_c.
struct ClientData {
  const void* x;     // [n, D] row-major; fp32, or bf16 when precision == 1
  const int32_t* y;  // [n]
  uint32_t n;
  uint32_t pad;
};

// What a local-SGD kernel leaves behind when a round's last sample is done:
// the device-side record of the event trigger (message (c, U_i, i)).
struct TriggerRec { uint32_t client, round, samples_done, flags; };
// What the aggregation kernel leaves behind per applied update.
struct ApplyRec { uint32_t client, round, h_after, seq; };

// Rows of the snapshot / update-sum / work arrays are `stride` floats apart
// (n_params rounded up to a multiple of 32, so every row is 128-byte aligned).
struct RoundLaunch {
  const TaskDesc* tasks;         // device
  const InflightRef* inflight;   // device
  const ClientData* clients;     // device, [n_clients]
  const uint64_t* sample_keys;   // device, [n_clients]
  const float* snaps;            // [n_snap, stride] models rounds start from
  float* U;                      // [n_u_rows, stride] update sums, row = TaskDesc::u_row
  float* w_end;                  // optional [n_events, stride] end-of-round models
  TriggerRec* trig;              // [n_events], row = seq
  uint32_t* status;              // optional: bit 0 set if a bounded device wait gave up,
                                 // bit 2 if a debug index check failed (see debug_checks)
  uint32_t debug_checks;         // non-zero: sample indices and row numbers are range-checked before use
  size_t stride;
  uint32_t task_begin, n_tasks;
  uint32_t n_u_rows, n_snap;     // extents of U and snaps (for the debug checks)
  uint32_t crowded_hint;         // non-zero: pick the kernel a full wave of this run's clients would get,
                                 // however few tasks this launch holds (single-task parity runs)
  uint32_t step_by_step;         // non-zero: the recurrence of a block is always walked step by step
  float l2;
};

// One CTA waits (at most max_polls polls) on a barrier nobody signals, then sets bit 0 of *status.
cudaError_t launch_wait_probe(uint32_t* status, uint32_t max_polls, cudaStream_t s);

// Softmax regression 784 -> 10, batch 1: one CTA per round-task; the kernel is picked by lambda and by
// how many round-tasks the launch holds.  Asynchronous on s; may start under the tail of the previous kernel in s
// (programmatic stream serialisation) and waits on the device before reading that kernel's output.
cudaError_t launch_lr_rounds(const RoundLaunch& p, cudaStream_t s);
// lambda = 0, more round-tasks than SMs: update sum in tensor memory, accumulated by tcgen05.mma (tf32 x 3)
bool lr_tc_eligible(const RoundLaunch& p);
cudaError_t launch_lr_tc_rounds(const RoundLaunch& p, cudaStream_t s);

struct MlpShape {
  uint32_t n_layers, dims[8], batch, precision;
  uint32_t cluster;              // CTAs per round-task
};
struct MlpLaunch {
  RoundLaunch r;
  MlpShape shape;
  float* work;                   // [n_clients, stride] client's current model
  float* act;                    // per-task activation scratch
  size_t act_stride;             // floats per task
};
cudaError_t launch_mlp_rounds(const MlpLaunch& p, cudaStream_t s);
size_t mlp_act_floats(const MlpShape& shape);
uint32_t mlp_pick_cluster(const MlpShape& shape, uint32_t n_clients);
const char* mlp_check_shape(const MlpShape& shape);  // null if the kernel can run it
// fp32 784-128-C models, batch 32: the model stays on-chip for the whole round (4-CTA cluster)
bool mlp_res_eligible(const MlpLaunch& p);
cudaError_t launch_mlp_res_rounds(const MlpLaunch& p, cudaStream_t s);
// bf16 D0-256-128-C models, batch 64: one CTA per round-task streams the first layer through a
// warp-specialised tcgen05 pipeline (see mlp_stream_kernel.cu)
bool mlp_stream_eligible(const MlpShape& shape);
cudaError_t launch_mlp_stream_rounds(const MlpLaunch& p, cudaStream_t s);
// bf16 models whose first layer fits the tensor-core kernel (tcgen05 + TMEM)
bool mlp_tc_eligible(const MlpShape& shape);
cudaError_t launch_mlp_tc_rounds(const MlpLaunch& p, cudaStream_t s);

// Small convolutional classifier (two 5x5 convolutions with average pooling, three dense layers):
// dims = {side, c_in, c1, c2, f1, f2, classes}; the whole model stays in shared memory for the round.
struct CnnShape { uint32_t dims[8], batch; };
struct CnnLaunch {
  RoundLaunch r;
  CnnShape shape;
  float* act;                    // per-task activation scratch
  size_t act_stride;             // floats per task
  uint32_t stage_rows = 0;       // set by the launcher: the CTA's minibatch rows fit in shared memory beside the model,
  uint32_t stage_acts = 0;       //   and so do its activations other than the first convolution's maps
};
uint32_t cnn_n_params(const CnnShape& s);
size_t cnn_act_floats(const CnnShape& s);
const char* cnn_check_shape(const CnnShape& s);   // null if the kernel can run it
cudaError_t launch_cnn_rounds(const CnnLaunch& p, cudaStream_t s);

// Ordered aggregation: for seq in [lo, hi): w -= eta_seq * U[seq]; keep a copy
// where a later round starts from it; bump H and log the apply.
struct ApplyLaunch {
  const ApplyDesc* applies;  // device, indexed by seq
  const float* U;
  float* snaps;
  const float* w_in;         // server model before the range [stride]
  float* w_out;              // ... and after it (may equal w_in only when groups == 1)
  float* totals;             // scratch [groups, stride], used when groups > 1
  uint32_t* H;               // [n_clients]
  ApplyRec* log;             // [n_events]
  uint32_t* status;          // optional: bit 1 set if the model after the range is not finite
  size_t stride;
  uint32_t n_params, lo, hi;
  uint32_t groups;           // apply_groups(hi - lo)
};
uint32_t apply_groups(uint32_t n_updates);
cudaError_t launch_apply_updates(const ApplyLaunch& p, cudaStream_t s);

// Peer-to-peer ring: the models of the nodes listed in applies[lo, hi) take their operations.
struct RingApplyLaunch {
  const RingApplyDesc* applies;  // device
  const RingOp* ops;             // device
  const float* U;                // [n_tasks, stride]
  float* node_w;                 // [n_nodes, stride]
  uint32_t* status;              // optional: bit 1 set if a model is not finite afterwards
  size_t stride;
  uint32_t n_params, lo, hi;
};
cudaError_t launch_ring_apply(const RingApplyLaunch& p, cudaStream_t s);

// Debug checks at load time: labels in range (else bit 2 of *status), pixels finite (else bit 1; x may be null).
cudaError_t launch_validate_data(const float* x, const int32_t* y, uint32_t n, uint32_t dim, uint32_t n_classes,
                                 uint32_t* status, cudaStream_t s);

#if defined(__CUDACC__)
// Debug check at the top of every round kernel (all threads of a CTA, and all CTAs of a cluster,
// take the same decision): are the rows and slots the task names inside the arrays?  If not,
// bit 2 of *status is set and the caller skips the task without touching memory.
__device__ __forceinline__ bool debug_task_ok(const RoundLaunch& p, const TaskDesc& t) {
  if (!p.debug_checks) return true;
  bool ok = t.u_row < p.n_u_rows && t.snap_slot < p.n_snap;
  for (uint32_t f = 0; ok && f < t.inflight_cnt; ++f) ok = p.inflight[t.inflight_off + f].row < p.n_u_rows;
  if (!ok && threadIdx.x == 0 && p.status) atomicOr(p.status, 4u);
  return ok;
}
// A round without a single iteration (a node the Setup split of Algorithm 2 gave nothing in this
// round): Algorithm 3 still sends (c, U_i, i) after the empty inner loop, with U_i = 0.  One CTA
// writes the zero update sum, the unchanged model where the caller wants it, and the trigger record.
__device__ __forceinline__ void publish_empty_round(const RoundLaunch& p, const TaskDesc& t, uint32_t n_params) {
  float* U = p.U + (size_t)t.u_row * p.stride;
  const float* snap = p.snaps + (size_t)t.snap_slot * p.stride;
  for (uint32_t i = threadIdx.x; i < n_params; i += blockDim.x) {
    U[i] = 0.f;
    if (p.w_end) {
      float w = snap[i];
      for (uint32_t f = 0; f < t.inflight_cnt; ++f) {
        const InflightRef ref = p.inflight[t.inflight_off + f];
        w = fmaf(-ref.eta, p.U[(size_t)ref.row * p.stride + i], w);
      }
      p.w_end[(size_t)t.u_row * p.stride + i] = w;
    }
  }
  if (threadIdx.x == 0) {
    TriggerRec rec;
    rec.client = t.client; rec.round = t.round; rec.samples_done = 0; rec.flags = 1;
    p.trig[t.seq] = rec;
  }
}
#endif

// bf16 conversion of a client's rows at load time (precision 1).
cudaError_t launch_to_bf16(const float* src, void* dst, size_t n, cudaStream_t s);

}  // namespace aet
