/*
 * aet.h - C ABI of the AET-SGD hot-path library for NVIDIA B200 (sm_100a).
 *
 * AET-SGD (asynchronous event-triggered SGD, arXiv 2112.13935): every client
 * runs local-SGD rounds whose length grows linearly, s_i = a*i + b (Section 5,
 * "Objective function"; Appendix Table 2), accumulates the update sum U_i of
 * the round's gradients and sends (c, U_i, i) when the round's last sample is
 * done - that is the event trigger (Algorithm 3, MainComputeNode).  A server
 * applies w -= eta_k * U in arrival order (Algorithm 3, Receive; Section 1,
 * client-server form) and clients pick the refreshed model up at their next
 * round start, subject to the delay checkpoint Synchronize(H, d, i).  Compute
 * and network delays are simulated (Section 3.3.2, Section 5 "System delay")
 * with a seeded integer clock, so the asynchronous interleaving is reproducible.
 *
 * All clients run concurrently on one GPU.  Every call returns an aet_status;
 * nothing throws, aborts or traps.  Out-parameters are untouched on error.
 * Unless a parameter says otherwise, "device pointer" means memory of the
 * current CUDA device and "host pointer" ordinary (pageable or pinned) memory.
 *
 * Parameter-vector layout (models, update sums): layers in order, each W_l
 * row-major [in, out] followed by b_l [out]; fp32.
 */
#ifndef AET_H_
#define AET_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct aet_handle aet_handle; /* opaque; owned by the library */

typedef enum {
  AET_OK = 0,
  AET_ERR_ARG = 1,     /* null / out-of-range argument                      */
  AET_ERR_CONFIG = 2,  /* configuration the library cannot run               */
  AET_ERR_STATE = 3,   /* call out of order, or device bookkeeping mismatch  */
  AET_ERR_NOMEM = 4,   /* host or device allocation failed                   */
  AET_ERR_CUDA = 5,    /* a CUDA runtime call failed (see aet_last_error)    */
  AET_ERR_TIMEOUT = 6, /* a bounded device-side wait gave up                 */
  AET_ERR_NUMERIC = 7  /* non-finite value met in the server model or in data */
} aet_status;

#define AET_MAX_LAYERS 7
#define AET_NEVER_WAIT 0xFFFFFFFFu /* max_lag_d: the checkpoint never blocks */
#define AET_TICKS_PER_UNIT (1u << 20)

/* Run configuration.  Plain data; struct_size = sizeof(aet_config). */
typedef struct {
  uint32_t struct_size;
  uint32_t n_clients;
  uint32_t model;      /* 0 = softmax regression, 1 = ReLU MLP (Eq. 1: f(w; xi)), 2 = a
                          small convolutional classifier of the LeNet shape (the paper's
                          model for its 28x28 sets): 5x5 valid convolution + ReLU + 2x2
                          average pooling, twice, then three dense layers           */
  uint32_t n_layers;   /* entries of dims - 1                                      */
  uint32_t dims[8];    /* {784,10}, {784,128,10}, {3072,256,128,10}; model 2:
                          {side, c_in, c1, c2, f1, f2, classes} = {28,1,6,16,120,84,10};
                          rows of a data set are then side*side*c_in values, plane by
                          plane, and parameters run W1[c1][c_in][5][5], b1,
                          W2[c2][c1][5][5], b2, then the dense layers as below      */
  uint32_t precision;  /* 0 = fp32; 1 = bf16 operands, fp32 accumulate and master */
  uint32_t batch;      /* samples per SGD iteration; must divide every s_i        */
  uint32_t sched_a, sched_b; /* s_i = a*i + b (Section 5; Table 2)                */
  uint32_t round_base; /* index of a client's first round                         */
  uint32_t max_lag_d;  /* threshold d of Synchronize (Algorithm 3)                */
  float lr, lr_beta;   /* eta_i = lr / (1 + lr_beta * sqrt(t)) (Section 5)        */
  float l2;            /* lambda of (lambda/2)|W|^2 on weight matrices            */
  uint32_t delay_dist; /* 0 = exponential(mean), 1 = uniform[lo, hi]: the paper draws
                          its delays uniformly (Section 5 "System delay", Appendix
                          "Hyper-parameters selection"); the exponential form and the
                          lo / hi fields below extend that to other delay models     */
  uint64_t seed;
  double compute_delay_mean, network_delay_mean; /* time units, dist 0           */
  double compute_delay_lo, compute_delay_hi;     /* time units, dist 1           */
  double network_delay_lo, network_delay_hi;
  double straggler_factor; /* scales the compute delay of the stragglers          */
  uint32_t n_stragglers;   /* the last n_stragglers client ids                    */
  uint32_t flags;          /* AET_FLAG_* bits, 0 for the defaults                  */
  uint32_t split_mode;     /* 0: every node runs its own sequence s_{i,c} = a*i + b (the
                              paper's experiments, Appendix A.2).  1: Algorithm 2, Setup:
                              s_i = a*i + b is the global size of round i and each of its
                              iterations goes to node c with probability p_c, so that
                              s_{i,c} = |{t : a(i,t) = c}| and E[s_{i,c}] = p_c s_i; needs
                              batch 1; a node that gets no iteration sends U = 0          */
  uint32_t topology;       /* 0: client-server (Section 1, Fig. 1a): a server applies the
                              sums and clients pull its model.  1: peer-to-peer ring (Fig. 1b,
                              the paper's experiments): every node keeps its own model and
                              history map, sends its sums to its two ring neighbours only
                              (no forwarding) and Synchronize looks at those neighbours     */
  const uint32_t* client_shares; /* split_mode 1: host array of n_clients integer weights,
                              p_c = shares[c] / sum (copied by aet_create); NULL: p_c = 1/n */
} aet_config;

/* aet_load_client_data keeps the caller's device pointers instead of copying
 * (precision 0 only; precision 1 always makes its own bf16 copy).  Both arrays
 * must be device memory, x 16-byte aligned with dims[0] a multiple of 4, and
 * must stay alive and unchanged until aet_destroy. */
#define AET_FLAG_BORROW_DATA 1u
/* Debug checks in place of a memory checker: every label is range-checked and
 * every pixel checked finite as a data set is loaded, and every round kernel
 * checks the rows and slots its task names before touching them.  A violation
 * sets a status word (nothing traps); the next synchronising call returns
 * AET_ERR_STATE or AET_ERR_NUMERIC and the task concerned was skipped. */
#define AET_FLAG_DEBUG_CHECKS 2u
/* Keep every round's update sum U_i until the next aet_run_rounds so that
 * aet_get_update_sum can read it back.  Without it the rows are recycled as
 * soon as the server has applied them (memory ~ rounds in flight, not all
 * rounds of the call). */
#define AET_FLAG_KEEP_UPDATE_SUMS 4u
/* Softmax regression with many clients takes eight steps of the recursion at
 * once and, where the coupling eta * (x_s . x_t) between them is small, solves
 * for the eight logit vectors by sweeps that stop when they no longer move
 * (2e-7).  This flag makes the kernel always walk the eight steps one after
 * the other instead (same result up to that tolerance; slower). */
#define AET_FLAG_STEPWISE_RECURRENCE 8u

/* One round-task = one message (c, U_i, i) of Algorithm 3.  64 bytes.
 * Times are integer ticks (2^20 per time unit).  In the ring topology a record
 * is one delivery (sender, round, destination): t_apply is its arrival, seq its
 * place among all deliveries ordered by (arrival, destination, sender, round),
 * seen the messages the SENDER had received when that round started. */
typedef struct {
  uint64_t t_start;    /* round began (after any checkpoint wait)                  */
  uint64_t t_trigger;  /* h reached s_{i,c}: the update sum was sent               */
  uint64_t t_apply;    /* the server applied it                                     */
  uint64_t wait_ticks; /* time spent blocked in Synchronize before t_start         */
  uint32_t client, round;
  uint32_t samples;    /* s_{i,c}                                                   */
  uint32_t steps;      /* SGD iterations = samples / batch                          */
  uint32_t seq;        /* position in the server's apply order                      */
  uint32_t seen;       /* updates already in the server model the round started from */
  uint32_t lag;        /* max(0, rounds done - min over other clients of H) at start */
  uint32_t dest;       /* ring: the node this delivery went to (0xFFFFFFFF: the node has
                          no neighbour); client-server: 0, the server                  */
} aet_event;

typedef struct {
  uint64_t messages_up;            /* update sums sent = events                    */
  uint64_t model_pulls;            /* round starts                                  */
  uint64_t samples_total;
  uint64_t messages_if_per_sample; /* one message per SGD iteration instead         */
  uint64_t messages_if_constant_b; /* constant round size s = first round's size    */
  uint64_t t_end_ticks;            /* simulated time of the last apply              */
} aet_summary;

/* Counters of the most recent aet_run_rounds (device times only when kernel
 * timing is on).  kernel ids: 0 local-SGD, 1 ordered aggregation. */
typedef struct {
  uint64_t waves;              /* groups of independent round-tasks launched        */
  uint64_t launches[4];        /* kernel launches per kernel id                     */
  double kernel_ms[4];         /* summed device time per kernel id                  */
  double plan_ms;              /* host time spent on schedule + launch plan         */
} aet_stats;

/* Create a run: n clients with local data sets and a server holding the global
 * model (Section 1, client-server form; Algorithm 2 "Setup" fixes the step-size
 * and sample-size sequences and d, here through cfg).  Allocates the global
 * model (zeros) and per-client state on the current CUDA device.  Errors: AET_ERR_ARG (null, bad struct_size),
 * AET_ERR_CONFIG (unsupported model/dims/batch), AET_ERR_CUDA, AET_ERR_NOMEM. */
aet_status aet_create(const aet_config* cfg, aet_handle** out);

/* End of the run of Algorithm 3's loop "for round i": free everything the
 * handle owns (synchronises the device first). */
aet_status aet_destroy(aet_handle* h);

/* Back to the state right after aet_create + aet_set_global_model + data load:
 * global model = the last model set (zeros if none), no rounds done, clock 0,
 * empty log.  Client data and cached schedules are kept. */
aet_status aet_reset(aet_handle* h, void* cuda_stream);

/* Set the server's model w_0 (Algorithm 2: "Initialize global model").
 * w0: host or device pointer, n_params floats in the layout above. */
aet_status aet_set_global_model(aet_handle* h, const float* w0, size_t n_params,
                                void* cuda_stream);

/* Give client `client` its local data set D_c (Section 1).  x: host or device
 * pointer, row-major [n, dims[0]] fp32; y: host or device pointer, [n] int32
 * class ids in [0, dims[last]).  The library copies (precision 1: converts to
 * bf16 once); the caller may free its buffers once `cuda_stream` has completed.
 * Errors: AET_ERR_ARG (client out of range, n == 0, n < batch, null). */
aet_status aet_load_client_data(aet_handle* h, uint32_t client, const void* x,
                                const int32_t* y, uint32_t n, void* cuda_stream);

/* Run n_rounds more rounds of every client (Algorithm 3, MainComputeNode loop
 * "for round i") with all update sums applied by the server (Receive), to
 * quiescence.  Asynchronous on `cuda_stream`; host work = the integer schedule
 * and the launch plan.  Errors: AET_ERR_STATE (a client has no data),
 * AET_ERR_CONFIG (batch does not divide s_i), AET_ERR_CUDA, AET_ERR_NOMEM. */
aet_status aet_run_rounds(aet_handle* h, uint32_t n_rounds, void* cuda_stream);

/* Optional: start computing, on a host thread of the library, what the next
 * aet_run_rounds(h, n_rounds) does on the host - the integer schedule of start,
 * trigger and apply times (Section 3.3.2 delays; Algorithm 3, Synchronize) and
 * the launch plan - so that it overlaps the caller's aet_load_client_data
 * copies.  Returns at once.  The result is used only if the handle's state is
 * the one it was computed for (otherwise aet_run_rounds computes its own); a
 * schedule error is reported by aet_run_rounds, not here.  aet_run_rounds,
 * aet_reset, aet_debug_run_client_round and aet_destroy wait for the thread.
 * Errors: AET_ERR_ARG (null), AET_ERR_STATE (no thread could be started). */
aet_status aet_prepare_rounds(aet_handle* h, uint32_t n_rounds);

/* Copy the server's model out: the global model w the server keeps and
 * broadcasts (Section 1; Algorithm 3, Receive: w = w - eta_k U).  Host or device
 * pointer, n_params floats.  Synchronises `cuda_stream`.  Errors:
 * AET_ERR_TIMEOUT, AET_ERR_STATE (debug check), AET_ERR_NUMERIC (a non-finite
 * value reached the model); `out` is then untouched and the handle stays usable
 * (aet_reset, reload the offending data, run again). */
aet_status aet_get_global_model(aet_handle* h, float* out, size_t n_params,
                                void* cuda_stream);

/* The model node `node` holds (host or device pointer, n_params floats): its
 * own model in the ring topology (Section 1, Fig. 1b: every compute node keeps
 * a model; at quiescence it is w_0 minus the applied sums of the node and of its
 * two neighbours); in the client-server topology the model every client would
 * pull, i.e. the server's.  Synchronises `cuda_stream`. */
aet_status aet_get_node_model(aet_handle* h, uint32_t node, float* out, size_t n_params,
                              void* cuda_stream);

/* The event log of all rounds run so far - one record per message (c, U_i, i)
 * of Algorithm 3 with its start, trigger and apply times, the checkpoint wait
 * (Synchronize) and the history count behind it - ordered by seq within each
 * aet_run_rounds call, and its summary (message counts for the communication-
 * cost comparison of Section 5).  `out` is a host array of `capacity`
 * records (may be null with capacity 0 to query *n_events).  Synchronises the
 * last stream used and cross-checks the trigger/apply records the kernels
 * wrote against the schedule (AET_ERR_STATE on a mismatch). */
aet_status aet_get_event_log(aet_handle* h, aet_event* out, size_t capacity,
                             size_t* n_events, aet_summary* summary);

/* Update sum number `seq` of the most recent aet_run_rounds (host or device
 * pointer, n_params floats).  Needs AET_FLAG_KEEP_UPDATE_SUMS (AET_ERR_STATE
 * without it: rows are recycled in both topologies).  In the ring topology
 * `seq` counts round-tasks in (trigger time, node, round) order.  Synchronises
 * `cuda_stream`. */
aet_status aet_get_update_sum(aet_handle* h, uint32_t seq, float* out, size_t n_params,
                              void* cuda_stream);

/* Parity aid, not part of a run: one round-task (client, round) of Algorithm 3
 * started from the caller's model w_in; writes the update sum U_i and the
 * client's end-of-round model (either may be null).  Pointers: host or device,
 * n_params floats each.  Uses the same sample indices the run would use.
 * Leaves the handle's state unchanged.  Synchronises `cuda_stream`. */
aet_status aet_debug_run_client_round(aet_handle* h, uint32_t client, uint32_t round,
                                      const float* w_in, float* U_out, float* w_out,
                                      void* cuda_stream);

/* Failure-detection aid: runs the give-up path of the kernels' bounded waits on
 * purpose.  One CTA polls a barrier that nothing signals at most max_polls times
 * (1 .. 2^24; a few milliseconds at most), flags the handle's device status word
 * as a round kernel would after a lost asynchronous copy, and returns normally.
 * The call synchronises `cuda_stream` and returns AET_ERR_TIMEOUT; the handle
 * and the CUDA context stay usable.  (The paper assumes messages are never lost,
 * Section 3.3.1; this guards the library's own asynchronous copies.) */
aet_status aet_debug_wait_probe(aet_handle* h, uint32_t max_polls, void* cuda_stream);

/* Record CUDA events around every kernel of later runs (adds a little launch
 * overhead) so that aet_get_stats can report device time per kernel. */
aet_status aet_set_kernel_timing(aet_handle* h, int enable);
aet_status aet_get_stats(aet_handle* h, aet_stats* out);

size_t aet_n_params(const aet_handle* h);

/* Text of the most recent error on this handle ("" if none); h may be null for
 * the last aet_create failure of the calling thread. */
const char* aet_last_error(const aet_handle* h);

/* One round-task with no handle and no allocation (the paper has no counterpart;
 * this serves callers that may not allocate device memory while they run, e.g.
 * a process whose memory was handed to a pool at start-up, or one that must keep
 * the device-wide synchronisation of cudaMalloc off its latency path).  It does
 * what aet_debug_run_client_round does for fp32 models: round `round` of client
 * `client` (Algorithm 3, MainComputeNode) from the model w_in, writing the update
 * sum U_out and the end-of-round model w_out.  x [n, dims[0]] fp32, y [n] int32,
 * w_in, U_out, w_out (n_params floats each) are DEVICE pointers owned by the
 * caller.  The entry point always runs the library's generic fp32 round kernel
 * (any layer widths; not the shape-specialised kernels a handle may pick), so
 * its results agree with aet_debug_run_client_round within fp32 rounding order,
 * not bit for bit.  The kernel's scratch (descriptors, the working model, activations)
 * is a fixed array inside the library image: every GPU that loads the library
 * holds about 1 MB for it until the process exits.  Limits: precision 0, at most
 * 131,072 parameters and 131,072 floats of activation scratch (about
 * 10 x batch x sum of layer widths); larger requests return AET_ERR_CONFIG
 * with the sizes in aet_last_error(NULL).  The call is asynchronous on
 * `cuda_stream`, launches two kernels and calls neither cudaMalloc nor
 * cudaFree.  Its first call on a device looks the array's device address up
 * (cudaGetSymbolAddress); make that first call outside any stream capture.
 * All calls share the one array and what the last call left in it (the entry
 * point clears what must start at zero), so two calls whose kernels could
 * overlap on the GPU - different streams, different threads - race: keep them
 * ordered on one stream or synchronise between them. */
aet_status aet_round_no_alloc(const aet_config* cfg, uint32_t client, uint32_t round,
                              const float* x, const int32_t* y, uint32_t n,
                              const float* w_in, float* U_out, float* w_out,
                              void* cuda_stream);

/* ---- host-only helpers (no GPU needed) -------------------------------- */

/* The integer schedule alone: what aet_run_rounds(n_rounds) on a fresh handle
 * would log.  Same record layout and ordering as aet_get_event_log. */
aet_status aet_schedule_only(const aet_config* cfg, uint32_t n_rounds, aet_event* out,
                             size_t capacity, size_t* n_events, aet_summary* summary);

/* Draw number `counter` of stream (seed, stream, client); streams: 0 sample
 * index, 1 compute delay, 2 network delay. */
uint64_t aet_debug_draw(uint64_t seed, uint32_t stream, uint32_t client, uint64_t counter);
/* Delay in ticks from a 64-bit draw: dist 0 -> exponential with mean p0 ticks,
 * dist 1 -> uniform on [p0, p1] ticks. */
uint64_t aet_debug_delay_ticks(uint32_t dist, uint64_t draw, uint64_t p0, uint64_t p1);
/* Number of waves (groups of mutually independent round-tasks) the launch
 * plan of a fresh run of n_rounds has; 0 on error. */
uint32_t aet_debug_plan_waves(const aet_config* cfg, uint32_t n_rounds);

/* The launch plan of a fresh run of n_rounds, for checking it on the host: tasks
 * in launch order (their seq, wave and the snapshot slot they start from; arrays
 * of n_clients * n_rounds entries), per seq the row of the update-sum array and
 * the slot the server model is kept in after that update (-1: none), the number
 * of updates applied after each wave (first counts[0] entries of an array of
 * n_clients * n_rounds), and counts = {waves, update-sum rows, snapshot slots}
 * the run allocates.  cfg->flags decides whether rows are recycled. */
aet_status aet_debug_plan_layout(const aet_config* cfg, uint32_t n_rounds, uint32_t* task_seq,
                                 uint32_t* task_wave, uint32_t* task_snap_slot, uint32_t* u_row,
                                 int32_t* snap_slot_after, uint32_t* apply_upto, uint32_t* counts);

#ifdef __cplusplus
}
#endif
#endif /* AET_H_ */
