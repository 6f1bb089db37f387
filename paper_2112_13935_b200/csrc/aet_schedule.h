// Host side of the hot path: the integer simulated-time schedule (which client
// triggers when, in which order the server applies the update sums) and the
// launch plan that groups independent round-tasks into waves.
#pragma once
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/aet.h"

namespace aet {

// Simulated-time state carried from one aet_run_rounds call to the next.
struct SchedState {
  uint64_t clock = 0;
  std::vector<uint32_t> H;  // updates of each client the server has applied
  uint32_t rounds_done = 0;
};

// Sum of a round's per-iteration compute delays and its network delay depend
// only on (client, round); cached so a repeated run does not redraw them.
struct DelayCache {
  std::vector<std::vector<uint64_t>> busy, net;  // [client][round - round_base]
  // Setup split (Algorithm 2), split_mode 1 only: s_{i,c} and its running sum per node
  std::vector<std::vector<uint32_t>> split;      // [client][round - round_base]
  std::vector<std::vector<uint64_t>> split_before;  // [client][round - round_base]: samples before that round
};

struct SchedResult {
  std::vector<aet_event> events;  // ordered by seq
  aet_summary summary;
};

uint32_t sample_size(const aet_config& c, uint32_t round);      // s_i = a i + b
uint64_t samples_before(const aet_config& c, uint32_t round);  // rounds round_base .. round-1
// The same per node: the node's own sequence, or (split_mode 1) its coin-flip share of the global
// round (Algorithm 2, Setup), which the cache must hold (ensure_split) for every round asked for.
void ensure_split(const aet_config& c, uint32_t last_round, DelayCache& cache);
uint32_t node_sample_size(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round);
uint64_t node_samples_before(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round);
// eta_0 / (1 + beta sqrt(t)), t = the node's own SGD iterations before the round (Section 4.1)
double round_step_size(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round);

// Returns false and fills err on an invalid configuration.
bool validate_config(const aet_config& c, std::string& err);
bool simulate(const aet_config& c, uint32_t n_rounds, SchedState& st, DelayCache& cache,
              SchedResult& out, std::string& err);

// ---- launch plan -------------------------------------------------------
struct TaskDesc {          // one round-task, read by the local-SGD kernels
  uint32_t client, round, seq;
  uint32_t snap_slot;      // snapshot of the server model the round starts from
  uint32_t n_samples, steps;
  uint32_t inflight_off, inflight_cnt;  // own update sums not yet applied at start
  uint64_t sample_ctr0;    // client's running sample counter at round start
  float eta;               // round step size
  uint32_t u_row;          // row of the update-sum array this round's U_i goes to
};
struct InflightRef { uint32_t row; float eta; };   // row of the update-sum array, step size of its round
struct ApplyDesc {         // one server update, in seq order
  float eta;
  int32_t snap_slot;       // where to keep the model after this update (-1: nowhere)
  uint32_t client, round;
  uint32_t u_row;          // row of the update-sum array that holds U of this update
};
struct Plan {
  std::vector<TaskDesc> tasks;       // sorted by wave, longest first inside a wave
  std::vector<uint32_t> wave_off;    // tasks of wave L: [wave_off[L], wave_off[L+1])
  std::vector<uint32_t> apply_upto;  // after wave L the server applies seq < apply_upto[L]
  std::vector<InflightRef> inflight;
  std::vector<ApplyDesc> applies;
  std::vector<uint32_t> u_row_of;    // seq -> row of the update-sum array
  uint32_t n_snap = 0;               // snapshot slots in use at once (slot 0 = model at call start)
  uint32_t n_u_rows = 0;             // update-sum rows in use at once
  uint32_t max_wave_tasks = 0;
};
// keep_all: one row per event and one slot per distinct start position, never reused
// (row = seq), so that every update sum can be read back after the run.  Otherwise rows
// and slots are recycled as soon as nothing later in the launch order reads them.
void build_plan(const aet_config& c, const DelayCache& cache, const std::vector<aet_event>& events, bool keep_all, Plan& plan);

// ---- peer-to-peer ring (Section 1, Fig. 1b) ------------------------------
// Every node keeps its own model and history map; a round's sum goes to the two ring neighbours
// only and is not forwarded.  One log record per delivery (sender, round, destination).
constexpr uint32_t kNoDest = 0xFFFFFFFFu;   // destination of the records of a node without neighbours
struct RingState {
  uint64_t clock = 0;
  std::vector<uint32_t> H;     // [2 * node + side]: messages node has received from that side's neighbour
  uint32_t rounds_done = 0;
};
struct RingTask {              // one round-task, in (t_trigger, client, round) order
  uint64_t t_start, t_trigger;
  uint32_t client, round, samples, steps;
  uint32_t applied_off, applied_cnt;   // deliveries (indices into RingResult::events) that reached the node
                                       // since its previous start, in arrival order
};
struct RingResult {
  std::vector<aet_event> events;       // deliveries ordered by seq; pad holds the destination
  std::vector<uint32_t> event_task;    // task index of the round each delivery carries
  std::vector<RingTask> tasks;
  std::vector<uint32_t> applied;       // flat lists referenced by RingTask
  aet_summary summary;
};
bool simulate_ring(const aet_config& c, uint32_t n_rounds, RingState& st, DelayCache& cache,
                   RingResult& out, std::string& err);

struct RingOp { uint32_t u_row; float eta; };   // w_node -= eta * U[u_row]
struct RingApplyDesc { uint32_t node, op_off, op_cnt, pad; };
struct RingPlan {
  std::vector<TaskDesc> tasks;          // sorted by wave; snap_slot = node, u_row = its row of the update-sum array, no sums in flight
  std::vector<uint32_t> wave_off;
  // before wave L (and once more after the last wave): the nodes whose models move and their operations
  std::vector<RingApplyDesc> applies;   // grouped by wave: [apply_off[L], apply_off[L + 1])
  std::vector<uint32_t> apply_off;      // n_waves + 2 entries
  std::vector<RingOp> ops;
  uint32_t max_wave_tasks = 0;
  uint32_t n_u_rows = 0;                // rows of the update-sum array the plan uses (rows are recycled unless keep_all)
};
void build_ring_plan(const aet_config& c, const DelayCache& cache, const RingResult& r, bool keep_all, RingPlan& plan);

}  // namespace aet
