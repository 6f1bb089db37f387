// Integer discrete-event schedule of AET-SGD and the wave plan built from it.
//
// Algorithm 3 (MainComputeNode): round i of client c runs s_{i,c} = a*i + b
// samples, then sends (c, U_i, i).  Section 3.3.2 / Section 5: every SGD
// iteration takes a random compute delay and every message a random network
// delay.  Receive bumps H_v per message; Synchronize(H, d, i) blocks a round
// start while (rounds done - min over the others of H) > d.  Ties in simulated
// time are broken by (tick, apply before start, client, round).
#include "aet_schedule.h"

#include <math.h>

#include <algorithm>
#include <queue>
#include <thread>
#include <tuple>

#include "aet_rng.h"

namespace aet {

uint32_t sample_size(const aet_config& c, uint32_t round) { return c.sched_a * round + c.sched_b; }

uint64_t samples_before(const aet_config& c, uint32_t round) {
  // sum_{j=base}^{round-1} (a j + b)
  uint64_t n = round - c.round_base;
  uint64_t sum_j = n * (uint64_t)c.round_base + n * (n - 1) / 2;
  return (uint64_t)c.sched_a * sum_j + (uint64_t)c.sched_b * n;
}

// Algorithm 2, Setup: iteration t of global round i goes to node a(i, t) = c with probability
// p_c = shares[c] / sum(shares) (all equal without shares); s_{i,c} counts the node's iterations.
// The coin of an iteration is draw number (iterations of all earlier rounds) + t of the stream
// (seed, setup, client 0); node = first c whose cumulative share exceeds hi32(draw) * sum >> 32.
void ensure_split(const aet_config& c, uint32_t last_round, DelayCache& cache) {
  if (!c.split_mode) return;
  const uint32_t n = c.n_clients;
  if (cache.split.size() != n) { cache.split.assign(n, {}); cache.split_before.assign(n, {}); }
  const uint32_t need = last_round - c.round_base;
  uint32_t have = (uint32_t)cache.split[0].size();
  if (have >= need) return;
  std::vector<uint64_t> cum(n);
  uint64_t total = 0;
  for (uint32_t cl = 0; cl < n; ++cl) { total += c.client_shares ? c.client_shares[cl] : 1u; cum[cl] = total; }
  const uint64_t key = stream_key(c.seed, kStreamSetup, 0);
  for (uint32_t rel = have; rel < need; ++rel) {
    const uint32_t round = c.round_base + rel;
    const uint64_t g0 = samples_before(c, round);
    const uint32_t s_i = sample_size(c, round);
    std::vector<uint32_t> cnt(n, 0);
    for (uint32_t t = 0; t < s_i; ++t) {
      const uint64_t v = ((draw(key, g0 + t) >> 32) * total) >> 32;
      const uint32_t cl = (uint32_t)(std::upper_bound(cum.begin(), cum.end(), v) - cum.begin());
      cnt[cl] += 1;
    }
    for (uint32_t cl = 0; cl < n; ++cl) {
      const uint64_t before = rel ? cache.split_before[cl][rel - 1] + cache.split[cl][rel - 1] : 0;
      cache.split[cl].push_back(cnt[cl]);
      cache.split_before[cl].push_back(before);
    }
  }
}

uint32_t node_sample_size(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round) {
  return c.split_mode ? cache.split[client][round - c.round_base] : sample_size(c, round);
}

uint64_t node_samples_before(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round) {
  return c.split_mode ? cache.split_before[client][round - c.round_base] : samples_before(c, round);
}

double round_step_size(const aet_config& c, const DelayCache& cache, uint32_t client, uint32_t round) {
  double t = (double)(node_samples_before(c, cache, client, round) / c.batch);
  return (double)c.lr / (1.0 + (double)c.lr_beta * sqrt(t));
}

static uint64_t to_ticks(double units) { return (uint64_t)floor(units * (double)AET_TICKS_PER_UNIT + 0.5); }

bool validate_config(const aet_config& c, std::string& err) {
  if (c.struct_size != sizeof(aet_config)) { err = "struct_size does not match this library's aet_config"; return false; }
  if (c.n_clients == 0) { err = "n_clients must be at least 1"; return false; }
  if (c.n_layers < 1 || c.n_layers > AET_MAX_LAYERS) { err = "n_layers out of range"; return false; }
  for (uint32_t l = 0; l <= c.n_layers; ++l)
    if (c.dims[l] == 0) { err = "a layer dimension is zero"; return false; }
  if (c.model > 2 || (c.model == 0 && c.n_layers != 1)) { err = "model 0 has exactly one weight layer"; return false; }
  if (c.model == 2 && (c.n_layers != 6 || c.precision != 0)) { err = "model 2 takes dims {side, c_in, c1, c2, f1, f2, classes} and precision 0"; return false; }
  if (c.precision > 1) { err = "precision must be 0 or 1"; return false; }
  if (c.batch == 0) { err = "batch must be at least 1"; return false; }
  if (c.delay_dist > 1) { err = "delay_dist must be 0 or 1"; return false; }
  if (c.n_stragglers > c.n_clients) { err = "more stragglers than clients"; return false; }
  if (!(c.lr > 0.f) || c.lr_beta < 0.f || c.l2 < 0.f) { err = "lr must be positive, lr_beta and l2 non-negative"; return false; }
  if (c.delay_dist == 0 && (!(c.compute_delay_mean >= 0) || !(c.network_delay_mean >= 0))) { err = "negative delay mean"; return false; }
  if (c.delay_dist == 1 && (c.compute_delay_hi < c.compute_delay_lo || c.network_delay_hi < c.network_delay_lo ||
                            c.compute_delay_lo < 0 || c.network_delay_lo < 0)) { err = "uniform delay range is empty"; return false; }
  if (!(c.straggler_factor >= 0) || c.straggler_factor > 65535.0) { err = "straggler_factor out of range"; return false; }
  if (c.split_mode > 1) { err = "split_mode must be 0 or 1"; return false; }
  if (c.topology > 1) { err = "topology must be 0 (client-server) or 1 (ring)"; return false; }
  if (c.split_mode && c.batch != 1) { err = "the Setup split assigns single SGD iterations: batch must be 1"; return false; }
  if (c.client_shares) {
    uint64_t total = 0;
    for (uint32_t cl = 0; cl < c.n_clients; ++cl) total += c.client_shares[cl];
    if (total == 0 || total > 0xFFFFFFFFull) { err = "client_shares must sum to 1 .. 2^32 - 1"; return false; }
  }
  return true;
}

namespace {

struct DelayModel {
  uint32_t dist;
  uint64_t c0, c1, n0, n1;  // dist 0: means; dist 1: lo / hi
  uint64_t straggler_q16;
  uint64_t compute(uint64_t r) const { return dist == 0 ? exp_ticks(r, c0) : uniform_ticks(r, c0, c1); }
  uint64_t network(uint64_t r) const { return dist == 0 ? exp_ticks(r, n0) : uniform_ticks(r, n0, n1); }
};

DelayModel make_delay_model(const aet_config& c) {
  DelayModel m;
  m.dist = c.delay_dist;
  if (c.delay_dist == 0) {
    m.c0 = to_ticks(c.compute_delay_mean); m.c1 = 0;
    m.n0 = to_ticks(c.network_delay_mean); m.n1 = 0;
  } else {
    m.c0 = to_ticks(c.compute_delay_lo); m.c1 = to_ticks(c.compute_delay_hi);
    m.n0 = to_ticks(c.network_delay_lo); m.n1 = to_ticks(c.network_delay_hi);
  }
  m.straggler_q16 = (uint64_t)floor(c.straggler_factor * 65536.0 + 0.5);
  return m;
}

// Fill cache.busy / cache.net for rounds [first, last) of every client.
void fill_delays(const aet_config& c, uint32_t first, uint32_t last, DelayCache& cache) {
  const uint32_t n = c.n_clients;
  if (cache.busy.size() != n) { cache.busy.assign(n, {}); cache.net.assign(n, {}); }
  const uint32_t need = last - c.round_base;
  bool missing = false;
  for (uint32_t cl = 0; cl < n; ++cl) missing |= cache.busy[cl].size() < need;
  if (!missing) return;
  const DelayModel dm = make_delay_model(c);
  auto work = [&](uint32_t cl) {
    const uint64_t kc = stream_key(c.seed, kStreamCompute, cl);
    const uint64_t kn = stream_key(c.seed, kStreamNetwork, cl);
    const bool straggler = cl >= n - c.n_stragglers;
    std::vector<uint64_t>& busy = cache.busy[cl];
    std::vector<uint64_t>& net = cache.net[cl];
    for (uint32_t rel = (uint32_t)busy.size(); rel < need; ++rel) {
      const uint32_t round = c.round_base + rel;
      const uint64_t it0 = node_samples_before(c, cache, cl, round) / c.batch;
      const uint32_t steps = node_sample_size(c, cache, cl, round) / c.batch;
      uint64_t sum = 0;
      for (uint32_t j = 0; j < steps; ++j) {
        uint64_t dt = dm.compute(draw(kc, it0 + j));
        if (straggler) { dt = (dt * dm.straggler_q16) >> 16; if (!dt) dt = 1; }
        sum += dt;
      }
      busy.push_back(sum);
      net.push_back(dm.network(draw(kn, round)));
    }
  };
  unsigned hw = std::thread::hardware_concurrency();
  unsigned nt = std::max(1u, std::min({hw ? hw : 1u, n, 32u}));
  if (nt == 1) { for (uint32_t cl = 0; cl < n; ++cl) work(cl); return; }
  std::vector<std::thread> pool;
  for (unsigned t = 0; t < nt; ++t)
    pool.emplace_back([&, t]() { for (uint32_t cl = t; cl < n; cl += nt) work(cl); });
  for (auto& th : pool) th.join();
}

enum Kind : uint32_t { kApply = 0, kStart = 1 };
struct QItem {
  uint64_t t; uint32_t kind, client, round;
  bool operator>(const QItem& o) const {
    return std::tie(t, kind, client, round) > std::tie(o.t, o.kind, o.client, o.round);
  }
};

}  // namespace

bool simulate(const aet_config& c, uint32_t n_rounds, SchedState& st, DelayCache& cache,
              SchedResult& out, std::string& err) {
  const uint32_t n = c.n_clients;
  if (st.H.size() != n) st.H.assign(n, 0);
  const uint32_t first = c.round_base + st.rounds_done, last = first + n_rounds;
  for (uint32_t r = first; r < last; ++r)
    if (sample_size(c, r) == 0 || sample_size(c, r) % c.batch) {
      err = "batch must divide every round's sample count, and rounds may not be empty";
      return false;
    }
  ensure_split(c, last, cache);
  fill_delays(c, first, last, cache);

  out.events.clear();
  out.events.reserve((size_t)n * n_rounds);
  std::vector<uint32_t>& H = st.H;
  std::vector<uint64_t> ready(n, st.clock);
  std::vector<int64_t> blocked(n, -1);  // round a client is waiting to start, or -1
  std::vector<uint32_t> ev_of((size_t)n * n_rounds);  // (client, round) -> index in out.events
  std::priority_queue<QItem, std::vector<QItem>, std::greater<QItem>> q;
  for (uint32_t cl = 0; cl < n && n_rounds; ++cl) q.push({st.clock, kStart, cl, first});
  const bool never_wait = c.max_lag_d == AET_NEVER_WAIT;
  uint32_t seq = 0, n_blocked = 0;

  auto lag_of = [&](uint32_t cl, uint32_t round) -> uint32_t {
    if (n == 1) return 0;
    uint32_t m = UINT32_MAX;
    for (uint32_t e = 0; e < n; ++e) if (e != cl && H[e] < m) m = H[e];
    uint32_t rel = round - c.round_base;
    return rel > m ? rel - m : 0;
  };

  while (!q.empty()) {
    QItem it = q.top();
    q.pop();
    if (it.kind == kApply) {
      H[it.client] += 1;
      out.events[ev_of[(size_t)it.client * n_rounds + (it.round - first)]].seq = seq++;
      if (n_blocked) {
        // min and second min of H once, then an O(1) test per blocked client
        uint32_t m1 = UINT32_MAX, m2 = UINT32_MAX, c1 = 0;
        for (uint32_t e = 0; e < n; ++e) {
          if (H[e] < m1) { m2 = m1; m1 = H[e]; c1 = 1; }
          else if (H[e] == m1) { ++c1; }
          else if (H[e] < m2) { m2 = H[e]; }
        }
        for (uint32_t b = 0; b < n; ++b) {
          if (blocked[b] < 0) continue;
          uint32_t mo = (H[b] == m1 && c1 == 1) ? m2 : m1;
          uint32_t rel = (uint32_t)blocked[b] - c.round_base;
          uint32_t lag = rel > mo ? rel - mo : 0;
          if (never_wait || lag <= c.max_lag_d) {
            q.push({it.t, kStart, b, (uint32_t)blocked[b]});
            blocked[b] = -1;
            --n_blocked;
          }
        }
      }
      continue;
    }
    const uint32_t cl = it.client, round = it.round;
    const uint32_t lag = lag_of(cl, round);
    if (!never_wait && lag > c.max_lag_d) { blocked[cl] = round; ++n_blocked; continue; }
    aet_event e;
    e.t_start = it.t;
    e.t_trigger = it.t + cache.busy[cl][round - c.round_base];
    e.t_apply = e.t_trigger + cache.net[cl][round - c.round_base];
    e.wait_ticks = it.t - ready[cl];
    e.client = cl; e.round = round;
    e.samples = node_sample_size(c, cache, cl, round);
    e.steps = e.samples / c.batch;
    e.seq = 0; e.seen = seq; e.lag = lag; e.dest = 0;
    ev_of[(size_t)cl * n_rounds + (round - first)] = (uint32_t)out.events.size();
    out.events.push_back(e);
    q.push({e.t_apply, kApply, cl, round});
    ready[cl] = e.t_trigger;
    if (round + 1 < last) q.push({e.t_trigger, kStart, cl, round + 1});
  }
  if (n_blocked || seq != out.events.size()) { err = "schedule did not reach quiescence"; return false; }
  std::sort(out.events.begin(), out.events.end(),
            [](const aet_event& a, const aet_event& b) { return a.seq < b.seq; });

  aet_summary& s = out.summary;
  s = aet_summary{};
  s.messages_up = s.model_pulls = out.events.size();
  for (const aet_event& e : out.events) s.samples_total += e.samples;
  s.messages_if_per_sample = s.samples_total / c.batch;
  uint64_t s_first = sample_size(c, c.round_base);
  if (c.split_mode) s_first = std::max<uint64_t>(1, s_first / n);   // a node's expected share of the first global round
  const uint64_t per_client = n ? s.samples_total / n : 0;
  s.messages_if_constant_b = s_first ? n * ((per_client + s_first - 1) / s_first) : 0;
  s.t_end_ticks = out.events.empty() ? st.clock : out.events.back().t_apply;
  st.clock = s.t_end_ticks;
  st.rounds_done += n_rounds;
  return true;
}

void build_plan(const aet_config& c, const DelayCache& cache, const std::vector<aet_event>& events, bool keep_all, Plan& plan) {
  const size_t E = events.size();
  plan = Plan{};
  plan.applies.resize(E);
  plan.u_row_of.assign(E, 0);
  // Level of a task = 1 + max(level of every update it starts from, level of
  // the client's previous round).  Tasks of one level are mutually independent.
  std::vector<uint32_t> order(E);
  for (size_t k = 0; k < E; ++k) order[k] = (uint32_t)k;
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    // an empty round starts and ends on the same tick as the client's next one: keep round order
    return std::tie(events[a].t_start, events[a].client, events[a].round) <
           std::tie(events[b].t_start, events[b].client, events[b].round);
  });
  std::vector<uint32_t> level(E, 0), prev_level(c.n_clients, 0);
  uint32_t pref = 0, pref_max = 0, n_waves = 0;
  for (uint32_t k : order) {
    const aet_event& e = events[k];
    while (pref < e.seen) { pref_max = std::max(pref_max, level[pref]); ++pref; }
    uint32_t lv = 1 + std::max(pref_max, prev_level[e.client]);
    level[k] = lv;
    prev_level[e.client] = lv;
    n_waves = std::max(n_waves, lv);
  }
  // Tasks grouped by wave, longest first.
  std::vector<uint32_t> by_wave(E);
  for (size_t k = 0; k < E; ++k) by_wave[k] = (uint32_t)k;
  std::sort(by_wave.begin(), by_wave.end(), [&](uint32_t a, uint32_t b) {
    if (level[a] != level[b]) return level[a] < level[b];
    if (events[a].samples != events[b].samples) return events[a].samples > events[b].samples;
    return a < b;
  });
  plan.wave_off.assign(n_waves + 1, 0);
  plan.apply_upto.assign(n_waves, 0);
  for (uint32_t k : by_wave) plan.wave_off[level[k]] += 1;   // size of wave level-1, shifted by one
  for (uint32_t L = 1; L <= n_waves; ++L) plan.wave_off[L] += plan.wave_off[L - 1];
  for (uint32_t L = 0; L < n_waves; ++L) {
    plan.max_wave_tasks = std::max(plan.max_wave_tasks, plan.wave_off[L + 1] - plan.wave_off[L]);
    // the next wave's tasks need every update with seq < their `seen`
    uint32_t upto = 0;
    if (L + 1 < n_waves) {
      for (uint32_t q = plan.wave_off[L + 1]; q < plan.wave_off[L + 2]; ++q)
        upto = std::max(upto, events[by_wave[q]].seen);
    } else {
      upto = (uint32_t)E;
    }
    plan.apply_upto[L] = std::max(upto, L ? plan.apply_upto[L - 1] : 0u);
  }
  // A client's update sums still in flight when one of its rounds starts.
  std::vector<std::vector<uint32_t>> mine(c.n_clients);
  for (size_t k = 0; k < E; ++k) mine[events[k].client].push_back((uint32_t)k);
  auto for_each_inflight = [&](const aet_event& e, auto&& fn) {
    for (uint32_t j : mine[e.client])
      if (events[j].round < e.round && events[j].seq >= e.seen) fn(j);
  };

  // ---- rows of the update-sum array and snapshot slots ----
  // Launch order: round kernel of wave 0, aggregation 0, round kernel of wave 1, ...  The row of
  // update k is written by the round kernel of its wave and last read by the later of the
  // aggregation that applies it and the round kernels of the tasks that start with it in flight.
  // The snapshot for start position v is written by the aggregation that applies update v - 1
  // and last read by the last wave holding a task with seen == v.
  std::vector<int32_t> slot_of(E + 1, -1);
  if (keep_all) {
    for (size_t k = 0; k < E; ++k) plan.u_row_of[k] = (uint32_t)k;
    plan.n_u_rows = (uint32_t)E;
    slot_of[0] = 0;
    plan.n_snap = 1;
    for (const aet_event& e : events) if (slot_of[e.seen] < 0) slot_of[e.seen] = (int32_t)plan.n_snap++;
  } else {
    std::vector<uint32_t> applied_in(E, 0), u_last(E, 0);
    {
      uint32_t lo = 0;
      for (uint32_t L = 0; L < n_waves; ++L) {
        for (uint32_t k = lo; k < plan.apply_upto[L]; ++k) applied_in[k] = L;
        lo = plan.apply_upto[L];
      }
    }
    std::vector<int32_t> snap_last(E + 1, -1);   // last wave reading the snapshot of position v
    for (size_t k = 0; k < E; ++k) {
      const uint32_t L = level[k] - 1;
      u_last[k] = std::max(u_last[k], applied_in[k]);
      snap_last[events[k].seen] = std::max(snap_last[events[k].seen], (int32_t)L);
      for_each_inflight(events[k], [&](uint32_t j) { u_last[j] = std::max(u_last[j], L); });
    }
    std::vector<std::vector<uint32_t>> u_dead_after(n_waves), snap_dead_after(n_waves);
    for (size_t k = 0; k < E; ++k) u_dead_after[u_last[k]].push_back((uint32_t)k);
    for (size_t v = 0; v <= E; ++v) if (snap_last[v] >= 0) snap_dead_after[snap_last[v]].push_back((uint32_t)v);
    std::vector<uint32_t> free_rows, free_slots;
    slot_of[0] = 0;            // written by the host before the first launch
    plan.n_snap = 1;
    uint32_t lo = 0;
    for (uint32_t L = 0; L < n_waves; ++L) {
      for (uint32_t q = plan.wave_off[L]; q < plan.wave_off[L + 1]; ++q) {   // round kernel of wave L writes
        const uint32_t k = by_wave[q];
        if (free_rows.empty()) { plan.u_row_of[k] = plan.n_u_rows++; }
        else { plan.u_row_of[k] = free_rows.back(); free_rows.pop_back(); }
      }
      // the round kernel of wave L has run when aggregation L writes: its snapshots are free
      for (uint32_t v : snap_dead_after[L]) free_slots.push_back((uint32_t)slot_of[v]);
      for (uint32_t k = lo; k < plan.apply_upto[L]; ++k) {                  // aggregation L writes
        const uint32_t v = k + 1;
        if (snap_last[v] < 0) continue;
        if (free_slots.empty()) { slot_of[v] = (int32_t)plan.n_snap++; }
        else { slot_of[v] = (int32_t)free_slots.back(); free_slots.pop_back(); }
      }
      lo = plan.apply_upto[L];
      for (uint32_t k : u_dead_after[L]) free_rows.push_back(plan.u_row_of[k]);
    }
  }

  for (size_t k = 0; k < E; ++k) {
    plan.applies[k].eta = (float)round_step_size(c, cache, events[k].client, events[k].round);
    plan.applies[k].snap_slot = slot_of[k + 1];
    plan.applies[k].client = events[k].client;
    plan.applies[k].round = events[k].round;
    plan.applies[k].u_row = plan.u_row_of[k];
  }
  plan.tasks.reserve(E);
  for (uint32_t k : by_wave) {
    const aet_event& e = events[k];
    TaskDesc t{};
    t.client = e.client; t.round = e.round; t.seq = e.seq;
    t.snap_slot = (uint32_t)slot_of[e.seen];
    t.n_samples = e.samples; t.steps = e.steps;
    t.sample_ctr0 = node_samples_before(c, cache, e.client, e.round);
    t.eta = (float)round_step_size(c, cache, e.client, e.round);
    t.u_row = plan.u_row_of[k];
    t.inflight_off = (uint32_t)plan.inflight.size();
    for_each_inflight(e, [&](uint32_t j) {
      plan.inflight.push_back({plan.u_row_of[j], (float)round_step_size(c, cache, events[j].client, events[j].round)});
    });
    t.inflight_cnt = (uint32_t)plan.inflight.size() - t.inflight_off;
    plan.tasks.push_back(t);
  }
}

// ---------------------------------------------------------------------------
// Peer-to-peer ring.  Algorithm 3 read per node: Receive bumps H_v[sender] when the message
// arrives, Synchronize(H, d, i) looks at the node's own neighbours, "Send a tuple (c, U_i, i) to
// the other c's neighbors" goes to the two ring neighbours with a network delay each (draw
// 2 * round + side of the sender's network stream; side 0 = node c - 1, side 1 = node c + 1).
// Ties: (tick, receive before start, node, then sender and round).
namespace {

struct RingQItem {
  uint64_t t; uint32_t kind, node, x, y;   // receive: node = destination, x = sender, y = round; start: x = round
  bool operator>(const RingQItem& o) const {
    return std::tie(t, kind, node, x, y) > std::tie(o.t, o.kind, o.node, o.x, o.y);
  }
};
enum RingKind : uint32_t { kReceive = 0, kRingStart = 1 };

// Neighbours of node c: up to two (side, node) pairs, no duplicates, never c itself.
int ring_neighbours(uint32_t n, uint32_t c, uint32_t (&side)[2], uint32_t (&node)[2]) {
  int cnt = 0;
  const uint32_t cand[2] = {(c + n - 1) % n, (c + 1) % n};
  for (uint32_t sd = 0; sd < 2; ++sd) {
    if (cand[sd] == c) continue;
    if (cnt == 1 && node[0] == cand[sd]) continue;
    side[cnt] = sd; node[cnt] = cand[sd]; ++cnt;
  }
  return cnt;
}

}  // namespace

bool simulate_ring(const aet_config& c, uint32_t n_rounds, RingState& st, DelayCache& cache,
                   RingResult& out, std::string& err) {
  const uint32_t n = c.n_clients;
  if (st.H.size() != 2 * (size_t)n) st.H.assign(2 * (size_t)n, 0);
  const uint32_t first = c.round_base + st.rounds_done, last = first + n_rounds;
  for (uint32_t r = first; r < last; ++r)
    if (sample_size(c, r) == 0 || sample_size(c, r) % c.batch) {
      err = "batch must divide every round's sample count, and rounds may not be empty";
      return false;
    }
  ensure_split(c, last, cache);
  fill_delays(c, first, last, cache);
  const DelayModel dm = make_delay_model(c);
  std::vector<uint64_t> key_n(n);
  for (uint32_t cl = 0; cl < n; ++cl) key_n[cl] = stream_key(c.seed, kStreamNetwork, cl);

  out = RingResult{};
  std::vector<uint32_t>& H = st.H;
  std::vector<uint64_t> ready(n, st.clock);
  std::vector<int64_t> blocked(n, -1);
  std::vector<std::vector<uint32_t>> pending(n);   // deliveries (creation index) that reached a node since its last start
  std::vector<uint32_t> n_received(n, 0);
  struct Made { aet_event e; uint32_t task_creation; bool sequenced; };
  std::vector<Made> made;                          // deliveries in creation order
  struct TaskTmp { RingTask t; std::vector<uint32_t> applied; };
  std::vector<TaskTmp> tmp;                        // tasks in start order
  std::priority_queue<RingQItem, std::vector<RingQItem>, std::greater<RingQItem>> q;
  for (uint32_t cl = 0; cl < n && n_rounds; ++cl) q.push({st.clock, kRingStart, cl, first, 0});
  const bool never_wait = c.max_lag_d == AET_NEVER_WAIT;
  uint32_t seq = 0, n_blocked = 0;
  // (destination, sender, round) -> creation index of the delivery
  std::vector<std::vector<uint32_t>> made_of((size_t)n * n_rounds);   // per sender task: its deliveries

  auto lag_of = [&](uint32_t cl, uint32_t round) -> uint32_t {
    uint32_t sd[2], nd[2];
    const int k = ring_neighbours(n, cl, sd, nd);
    if (!k) return 0;
    uint32_t m = UINT32_MAX;
    for (int j = 0; j < k; ++j) m = std::min(m, H[2 * cl + sd[j]]);
    const uint32_t rel = round - c.round_base;
    return rel > m ? rel - m : 0;
  };

  while (!q.empty()) {
    const RingQItem it = q.top();
    q.pop();
    if (it.kind == kReceive) {
      const uint32_t dest = it.node, sender = it.x, round = it.y;
      // which side of dest the sender sits on
      uint32_t sd[2], nd[2];
      const int k = ring_neighbours(n, dest, sd, nd);
      for (int j = 0; j < k; ++j) if (nd[j] == sender) H[2 * dest + sd[j]] += 1;
      for (uint32_t m : made_of[(size_t)sender * n_rounds + (round - first)])
        if (made[m].e.dest == dest && !made[m].sequenced) {
          made[m].e.seq = seq++;
          made[m].sequenced = true;
          pending[dest].push_back(m);
          break;
        }
      n_received[dest] += 1;
      if (blocked[dest] >= 0 && (never_wait || lag_of(dest, (uint32_t)blocked[dest]) <= c.max_lag_d)) {
        q.push({it.t, kRingStart, dest, (uint32_t)blocked[dest], 0});
        blocked[dest] = -1;
        --n_blocked;
      }
      continue;
    }
    const uint32_t cl = it.node, round = it.x;
    const uint32_t lag = lag_of(cl, round);
    if (!never_wait && lag > c.max_lag_d) { blocked[cl] = round; ++n_blocked; continue; }
    TaskTmp tt;
    tt.t.t_start = it.t;
    tt.t.t_trigger = it.t + cache.busy[cl][round - c.round_base];
    tt.t.client = cl; tt.t.round = round;
    tt.t.samples = node_sample_size(c, cache, cl, round);
    tt.t.steps = tt.t.samples / c.batch;
    tt.t.applied_off = tt.t.applied_cnt = 0;
    tt.applied.swap(pending[cl]);
    aet_event e{};
    e.t_start = it.t; e.t_trigger = tt.t.t_trigger; e.wait_ticks = it.t - ready[cl];
    e.client = cl; e.round = round; e.samples = tt.t.samples; e.steps = tt.t.steps;
    e.seen = n_received[cl]; e.lag = lag;
    uint32_t sd[2], nd[2];
    const int k = ring_neighbours(n, cl, sd, nd);
    const uint32_t task_creation = (uint32_t)tmp.size();
    for (int j = 0; j < k; ++j) {
      e.t_apply = tt.t.t_trigger + dm.network(draw(key_n[cl], 2ull * round + sd[j]));
      e.dest = nd[j];
      made_of[(size_t)cl * n_rounds + (round - first)].push_back((uint32_t)made.size());
      made.push_back({e, task_creation, false});
      q.push({e.t_apply, kReceive, nd[j], cl, round});
    }
    if (!k) {
      e.t_apply = tt.t.t_trigger;
      e.dest = kNoDest;
      made.push_back({e, task_creation, false});
    }
    tmp.push_back(std::move(tt));
    ready[cl] = e.t_trigger;
    if (round + 1 < last) q.push({e.t_trigger, kRingStart, cl, round + 1, 0});
  }
  if (n_blocked) { err = "schedule did not reach quiescence"; return false; }
  // records of a node without neighbours take their places by trigger time
  {
    std::vector<uint32_t> lone;
    for (uint32_t m = 0; m < made.size(); ++m) if (made[m].e.dest == kNoDest) lone.push_back(m);
    std::sort(lone.begin(), lone.end(), [&](uint32_t a, uint32_t b) {
      return std::tie(made[a].e.t_apply, made[a].e.client, made[a].e.round) <
             std::tie(made[b].e.t_apply, made[b].e.client, made[b].e.round);
    });
    for (uint32_t m : lone) { made[m].e.seq = seq++; made[m].sequenced = true; }
  }
  if (seq != made.size()) { err = "schedule did not deliver every message"; return false; }
  // tasks in (t_trigger, client, round) order; deliveries in seq order
  std::vector<uint32_t> torder(tmp.size());
  for (uint32_t k = 0; k < tmp.size(); ++k) torder[k] = k;
  std::sort(torder.begin(), torder.end(), [&](uint32_t a, uint32_t b) {
    return std::tie(tmp[a].t.t_trigger, tmp[a].t.client, tmp[a].t.round) <
           std::tie(tmp[b].t.t_trigger, tmp[b].t.client, tmp[b].t.round);
  });
  std::vector<uint32_t> task_index(tmp.size());
  for (uint32_t k = 0; k < torder.size(); ++k) task_index[torder[k]] = k;
  out.events.resize(made.size());
  out.event_task.resize(made.size());
  for (const Made& m : made) {
    out.events[m.e.seq] = m.e;
    out.event_task[m.e.seq] = task_index[m.task_creation];
  }
  out.tasks.resize(tmp.size());
  for (uint32_t k = 0; k < torder.size(); ++k) {
    TaskTmp& tt = tmp[torder[k]];
    tt.t.applied_off = (uint32_t)out.applied.size();
    tt.t.applied_cnt = (uint32_t)tt.applied.size();
    for (uint32_t m : tt.applied) out.applied.push_back(made[m].e.seq);
    out.tasks[k] = tt.t;
  }
  aet_summary& s = out.summary;
  s = aet_summary{};
  uint64_t links = 0;
  for (uint32_t cl = 0; cl < n; ++cl) { uint32_t sd[2], nd[2]; links += ring_neighbours(n, cl, sd, nd); }
  for (const aet_event& e : out.events) if (e.dest != kNoDest) s.messages_up += 1;
  for (const RingTask& t : out.tasks) s.samples_total += t.samples;
  s.model_pulls = 0;
  s.messages_if_per_sample = (s.samples_total / c.batch) * (n ? links / n : 0);
  uint64_t s_first = sample_size(c, c.round_base);
  if (c.split_mode) s_first = std::max<uint64_t>(1, s_first / n);
  const uint64_t per_client = n ? s.samples_total / n : 0;
  s.messages_if_constant_b = s_first ? links * ((per_client + s_first - 1) / s_first) : 0;
  s.t_end_ticks = st.clock;
  for (const aet_event& e : out.events) s.t_end_ticks = std::max(s.t_end_ticks, e.t_apply);
  st.clock = s.t_end_ticks;
  st.rounds_done += n_rounds;
  return true;
}

// Waves and per-node operation lists of a ring run.  A round-task's level is one more than the
// levels of its node's previous round and of every round whose sum reached the node before it
// started.  Before wave L the model of every node with a task in L takes, in this order, the
// node's own previous sum (the net effect of that round's inner loop) and the sums that arrived
// since its previous start; after the last wave every node takes what is still outstanding.
void build_ring_plan(const aet_config& c, const DelayCache& cache, const RingResult& r, bool keep_all, RingPlan& plan) {
  plan = RingPlan{};
  const uint32_t n = c.n_clients;
  const size_t T = r.tasks.size();
  std::vector<uint32_t> order(T);
  for (size_t k = 0; k < T; ++k) order[k] = (uint32_t)k;
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
    return std::tie(r.tasks[a].t_start, r.tasks[a].client, r.tasks[a].round) <
           std::tie(r.tasks[b].t_start, r.tasks[b].client, r.tasks[b].round);
  });
  std::vector<uint32_t> level(T, 0), prev_level(n, 0);
  std::vector<int64_t> prev_task(T, -1), last_task(n, -1);
  uint32_t n_waves = 0;
  for (uint32_t k : order) {
    const RingTask& t = r.tasks[k];
    uint32_t lv = prev_level[t.client];
    for (uint32_t a = 0; a < t.applied_cnt; ++a) lv = std::max(lv, level[r.event_task[r.applied[t.applied_off + a]]]);
    level[k] = lv + 1;
    prev_level[t.client] = lv + 1;
    prev_task[k] = last_task[t.client];
    last_task[t.client] = k;
    n_waves = std::max(n_waves, lv + 1);
  }
  std::vector<uint32_t> by_wave(T);
  for (size_t k = 0; k < T; ++k) by_wave[k] = (uint32_t)k;
  std::sort(by_wave.begin(), by_wave.end(), [&](uint32_t a, uint32_t b) {
    if (level[a] != level[b]) return level[a] < level[b];
    if (r.tasks[a].samples != r.tasks[b].samples) return r.tasks[a].samples > r.tasks[b].samples;
    return a < b;
  });
  plan.wave_off.assign(n_waves + 1, 0);
  for (uint32_t k : by_wave) plan.wave_off[level[k]] += 1;
  for (uint32_t L = 1; L <= n_waves; ++L) plan.wave_off[L] += plan.wave_off[L - 1];
  plan.apply_off.assign(n_waves + 2, 0);
  std::vector<char> delivered(r.events.size(), 0);
  auto eta_of_task = [&](uint32_t k) { return (float)round_step_size(c, cache, r.tasks[k].client, r.tasks[k].round); };
  for (uint32_t L = 0; L < n_waves; ++L) {
    plan.max_wave_tasks = std::max(plan.max_wave_tasks, plan.wave_off[L + 1] - plan.wave_off[L]);
    for (uint32_t q = plan.wave_off[L]; q < plan.wave_off[L + 1]; ++q) {
      const uint32_t k = by_wave[q];
      const RingTask& t = r.tasks[k];
      TaskDesc d{};
      d.client = t.client; d.round = t.round; d.seq = k; d.snap_slot = t.client;
      d.n_samples = t.samples; d.steps = t.steps;
      d.inflight_off = 0; d.inflight_cnt = 0;
      d.sample_ctr0 = node_samples_before(c, cache, t.client, t.round);
      d.eta = eta_of_task(k);
      d.u_row = k;
      plan.tasks.push_back(d);
      RingApplyDesc a{t.client, (uint32_t)plan.ops.size(), 0, 0};
      if (prev_task[k] >= 0) plan.ops.push_back({(uint32_t)prev_task[k], eta_of_task((uint32_t)prev_task[k])});
      for (uint32_t j = 0; j < t.applied_cnt; ++j) {
        const uint32_t ev = r.applied[t.applied_off + j];
        plan.ops.push_back({r.event_task[ev], eta_of_task(r.event_task[ev])});
        delivered[ev] = 1;
      }
      a.op_cnt = (uint32_t)plan.ops.size() - a.op_off;
      if (a.op_cnt) plan.applies.push_back(a);
    }
    plan.apply_off[L + 1] = (uint32_t)plan.applies.size();
  }
  // Shift: the operations collected for wave L run before it, i.e. they belong to slot L.
  // apply_off[L] .. apply_off[L + 1] already has that meaning (slot 0 = before wave 0).
  // After the last wave: every node's last own sum and the deliveries nobody has taken yet, in seq order.
  std::vector<std::vector<RingOp>> tail(n);
  for (uint32_t cl = 0; cl < n; ++cl)
    if (last_task[cl] >= 0) tail[cl].push_back({(uint32_t)last_task[cl], eta_of_task((uint32_t)last_task[cl])});
  for (size_t ev = 0; ev < r.events.size(); ++ev)
    if (!delivered[ev] && r.events[ev].dest != kNoDest)
      tail[r.events[ev].dest].push_back({r.event_task[ev], eta_of_task(r.event_task[ev])});
  for (uint32_t cl = 0; cl < n; ++cl) {
    if (tail[cl].empty()) continue;
    RingApplyDesc a{cl, (uint32_t)plan.ops.size(), (uint32_t)tail[cl].size(), 0};
    plan.ops.insert(plan.ops.end(), tail[cl].begin(), tail[cl].end());
    plan.applies.push_back(a);
  }
  plan.apply_off[n_waves + 1] = (uint32_t)plan.applies.size();

  // Rows of the update-sum array.  Up to here tasks and operations name a sum by its round-task.  A sum is read
  // for the last time by the Receive step of some slot L (slot L runs before wave L; the slot after the last wave
  // takes what is left), so its row can be written again by a round-task of wave L or later.  keep_all: one row
  // per round-task, row = round-task (the caller wants to read the sums back).
  std::vector<uint32_t> row_of(T);
  if (keep_all) {
    for (size_t k = 0; k < T; ++k) row_of[k] = (uint32_t)k;
    plan.n_u_rows = (uint32_t)T;
  } else {
    std::vector<uint32_t> last_use(T, 0);
    for (uint32_t L = 0; L <= n_waves; ++L)
      for (uint32_t q = plan.apply_off[L]; q < plan.apply_off[L + 1]; ++q) {
        const RingApplyDesc& a = plan.applies[q];
        for (uint32_t o = 0; o < a.op_cnt; ++o) last_use[plan.ops[a.op_off + o].u_row] = L;   // slots ascend
      }
    std::vector<std::vector<uint32_t>> dies_at(n_waves + 1);
    for (size_t k = 0; k < T; ++k) dies_at[std::max(last_use[k], level[k])].push_back((uint32_t)k);
    std::vector<uint32_t> free_rows;
    uint32_t n_rows = 0;
    for (uint32_t L = 0; L < n_waves; ++L) {
      // sums whose last reader is slot L or earlier: slot L has run when wave L is launched
      for (uint32_t k : dies_at[L])
        if (last_use[k] <= L && level[k] - 1 < L) free_rows.push_back(row_of[k]);
      for (uint32_t q = plan.wave_off[L]; q < plan.wave_off[L + 1]; ++q) {
        const uint32_t k = by_wave[q];
        if (!free_rows.empty()) { row_of[k] = free_rows.back(); free_rows.pop_back(); }
        else row_of[k] = n_rows++;
      }
    }
    plan.n_u_rows = n_rows ? n_rows : 1;
  }
  for (TaskDesc& d : plan.tasks) d.u_row = row_of[d.u_row];
  for (RingOp& o : plan.ops) o.u_row = row_of[o.u_row];
}

}  // namespace aet
