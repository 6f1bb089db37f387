// aet_round_no_alloc: one round-task without a handle and without any allocation.
//
// Some hosts of this library may not allocate device memory while they run: a
// service that has handed all of its device memory to a pool at start-up, code
// running between a framework's allocator snapshots, or a process that must keep
// cudaMalloc (which synchronises the device) off its latency path.  For them the
// scratch the round kernel needs - the task and client descriptors, the client's
// working copy of the model and the per-task activation buffers - lives in a
// fixed array in device memory that is part of the library image.  Every GPU
// that loads the library holds these kMaxScratchBytes until the process exits.
#include <cuda_runtime.h>

#include <atomic>
#include <string>

#include "../../include/aet.h"
#include "aet_kernels.h"
#include "aet_rng.h"
#include "aet_schedule.h"

namespace aet {
void set_thread_error(const std::string& msg);  // text returned by aet_last_error(NULL)
}
using namespace aet;

namespace {

constexpr size_t kMaxParams = 131072;   // floats of the model (512 KB work row)
constexpr size_t kMaxActFloats = 131072;  // floats of activation scratch
constexpr size_t kHeaderBytes = 256;
constexpr size_t kMaxScratchBytes = kHeaderBytes + (kMaxParams + kMaxActFloats) * sizeof(float);

// The name below is a device symbol.  Host code never uses it as an address:
// it asks the runtime for the device address once per device (scratch_for).
static __device__ __align__(256) unsigned char g_scratch[kMaxScratchBytes];

// First kHeaderBytes of the scratch.  `status` is where the round kernel would flag a bounded
// wait that gave up; the generic fp32 kernel this entry point always runs has no such waits, and
// no call reads the word back.  A kernel with bounded waits must not be routed through here
// without adding that read.
struct Header {
  TaskDesc task;
  ClientData client;
  uint64_t key;
  TriggerRec trig;
  uint32_t status;
};
static_assert(sizeof(Header) <= kHeaderBytes, "header does not fit");

__global__ void fill_header_kernel(TaskDesc t, ClientData c, uint64_t key) {
  Header* h = reinterpret_cast<Header*>(g_scratch);
  h->task = t;
  h->client = c;
  h->key = key;
  h->trig = TriggerRec{0, 0, 0, 0};
  h->status = 0;
}

constexpr int kMaxDevices = 64;
std::atomic<unsigned char*> g_dev_ptr[kMaxDevices] = {};   // two host threads may look an address up at once: same value

// Device address of the scratch on the current device; looked up on first use.
cudaError_t scratch_for_current_device(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  unsigned char* known = g_dev_ptr[dev].load(std::memory_order_acquire);
  if (!known) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_scratch);
    if (e != cudaSuccess) return e;
    known = static_cast<unsigned char*>(p);
    g_dev_ptr[dev].store(known, std::memory_order_release);
  }
  *out = known;
  return cudaSuccess;
}

aet_status fail(aet_status s, const std::string& msg) {
  set_thread_error(msg);
  return s;
}

}  // namespace

extern "C" aet_status aet_round_no_alloc(const aet_config* cfg, uint32_t client, uint32_t round,
                                         const float* x, const int32_t* y, uint32_t n,
                                         const float* w_in, float* U_out, float* w_out,
                                         void* cuda_stream) {
  if (!cfg || !x || !y || !w_in || !U_out || !w_out) return fail(AET_ERR_ARG, "null argument");
  if (cfg->struct_size != sizeof(aet_config)) return fail(AET_ERR_ARG, "struct_size does not match sizeof(aet_config)");
  std::string err;
  if (!validate_config(*cfg, err)) return fail(AET_ERR_CONFIG, err);
  if (cfg->precision != 0) return fail(AET_ERR_CONFIG, "aet_round_no_alloc runs fp32 models only");
  if (cfg->model > 1) return fail(AET_ERR_CONFIG, "aet_round_no_alloc runs softmax regression and ReLU MLPs only");
  if (cfg->split_mode != 0) return fail(AET_ERR_CONFIG, "aet_round_no_alloc runs a node's own sequence s_i = a*i + b only (split_mode 0)");
  if (client >= cfg->n_clients) return fail(AET_ERR_ARG, "client index out of range");
  if (round < cfg->round_base) return fail(AET_ERR_ARG, "round is before round_base");
  if (n == 0 || n < cfg->batch) return fail(AET_ERR_ARG, "a client needs at least max(1, batch) samples");
  if (cfg->dims[cfg->n_layers] > 32) return fail(AET_ERR_CONFIG, "at most 32 classes are supported");
  const uint32_t s_i = sample_size(*cfg, round);
  if (s_i == 0 || s_i % cfg->batch) return fail(AET_ERR_CONFIG, "batch must divide the round's sample count");

  MlpShape shape{};
  shape.n_layers = cfg->n_layers;
  for (int i = 0; i < 8; ++i) shape.dims[i] = cfg->dims[i];
  shape.batch = cfg->batch;
  shape.precision = 0;
  shape.cluster = mlp_pick_cluster(shape, 1);
  if (const char* why = mlp_check_shape(shape)) return fail(AET_ERR_CONFIG, why);
  uint64_t P = 0;
  for (uint32_t l = 0; l < cfg->n_layers; ++l) P += (uint64_t)cfg->dims[l] * cfg->dims[l + 1] + cfg->dims[l + 1];
  const size_t act = mlp_act_floats(shape);
  if (P > kMaxParams || act > kMaxActFloats)
    return fail(AET_ERR_CONFIG, "model or batch too large for the fixed scratch of aet_round_no_alloc (" +
                                    std::to_string(kMaxParams) + " parameters, " + std::to_string(kMaxActFloats) +
                                    " activation floats); this one needs " + std::to_string(P) + " and " +
                                    std::to_string(act));

  unsigned char* base = nullptr;
  cudaError_t e = scratch_for_current_device(&base);
  if (e != cudaSuccess) { cudaGetLastError(); return fail(AET_ERR_CUDA, std::string("scratch lookup: ") + cudaGetErrorString(e)); }
  Header* hd = reinterpret_cast<Header*>(base);
  float* work = reinterpret_cast<float*>(base + kHeaderBytes);
  float* actp = work + kMaxParams;

  cudaStream_t s = (cudaStream_t)cuda_stream;
  TaskDesc t{};
  t.client = 0;  // the single descriptor in the scratch
  t.round = round; t.seq = 0; t.snap_slot = 0;
  t.n_samples = s_i; t.steps = s_i / cfg->batch;
  t.inflight_off = 0; t.inflight_cnt = 0;
  t.sample_ctr0 = samples_before(*cfg, round);
  t.eta = (float)round_step_size(*cfg, DelayCache{}, client, round);
  const ClientData cd{x, y, n, 0};
  fill_header_kernel<<<1, 1, 0, s>>>(t, cd, stream_key(cfg->seed, kStreamSample, client));
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(AET_ERR_CUDA, std::string("descriptor kernel: ") + cudaGetErrorString(e));

  MlpLaunch m{};
  m.r.tasks = &hd->task; m.r.inflight = nullptr; m.r.clients = &hd->client; m.r.sample_keys = &hd->key;
  m.r.snaps = w_in; m.r.U = U_out; m.r.w_end = w_out; m.r.trig = &hd->trig; m.r.status = &hd->status;
  m.r.stride = 0;  // one row everywhere: seq, snap_slot and client index are all 0
  m.r.task_begin = 0; m.r.n_tasks = 1; m.r.l2 = cfg->l2;
  m.shape = shape;
  m.work = work;
  m.act = actp;
  m.act_stride = act;
  e = launch_mlp_rounds(m, s);
  if (e != cudaSuccess) { cudaGetLastError(); return fail(AET_ERR_CUDA, std::string("round kernel: ") + cudaGetErrorString(e)); }
  return AET_OK;
}
