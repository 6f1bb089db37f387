"""Sample-size schedule, round step sizes and the simulated-time event schedule.

TEST INFRASTRUCTURE (see the package header).  Integer arithmetic only, apart
from the step size.

Follows the paper as below.
* Section 5 "Objective function" / Appendix Table 2: s_i = a * i^p + b with
  p = 1; the experiments give every node its own sequence s_{i,c} = a*i + b
  (Appendix A.2), which is the reading used here.
* Section 4.1: the step size is constant inside a round and diminishes as
  eta_0 / (1 + beta * sqrt(t)), t = iterations done before the round (here:
  the client's own count).
* Algorithm 3: a round ends (the event triggers) when the local counter h
  reaches s_{i,c}; the node then sends (c, U_i, i).  Receive applies
  w -= eta_k * U and bumps H_v.  Synchronize(H, d, i) blocks while
  max_e (i - H_e) > d.  Because H only grows and i is fixed within a round, the
  check can only block before the round's first iteration, so it is evaluated
  at round start.
* Section 3.3.2 / Section 5 "System delay": a random compute delay per SGD
  iteration and a random network delay per transmitted update sum.
Client-server form of Section 1: the server applies update sums in arrival
order; a client pulls the server's model when its round starts.

Conventions the paper leaves open (fixed here):
* time is integer ticks, 2^20 per unit; ties are ordered by
  (tick, APPLY before START, client, round);
* H_c counts the updates of client c the server has applied (Algorithm 3 bumps
  H_v once per message whatever its round), the maximum runs over e != c, and
  a lone client never waits;
* stragglers are the last n_stragglers client ids; their compute-delay draws
  are scaled by a Q16 fixed-point factor.
"""
import heapq
import math
import struct

from . import rng

APPLY, START = 0, 1
NEVER_WAIT = 0xFFFFFFFF
EVENT_STRUCT = struct.Struct("<4Q8I")   # layout of the library's event record


def sample_size(a: int, b: int, i: int) -> int:
    return a * i + b


def samples_before(a: int, b: int, base: int, i: int) -> int:
    """Samples a client has consumed before round i (rounds base .. i-1)."""
    return sum(sample_size(a, b, j) for j in range(base, i))


def rounds_needed(K: int, a: int, b: int, base: int) -> int:
    """Smallest T with s_base + ... + s_{base+T-1} >= K (Section 4.1: K = sum s_j)."""
    total, T = 0, 0
    while total < K:
        total += sample_size(a, b, base + T)
        T += 1
    return T


def round_step_size(lr: float, beta: float, t: int) -> float:
    return lr / (1.0 + beta * math.sqrt(t))


# ---- Algorithm 2, "Setup": the coin-flip split of a global round size among the nodes ----
# With cfg["split_mode"] == 1 the sequence s_i = a*i + b is the GLOBAL number of SGD iterations
# of round i; each of its iterations t is assigned to node c with probability p_c
# (a(i, t) = c) and s_{i,c} = |{t : a(i, t) = c}|, so E[s_{i,c}] = p_c s_i.  p_c is given by
# integer shares (p_c = shares[c] / sum(shares); all equal when absent: the paper's p_c = 1/n).
# The coin of iteration t of round i is draw number (iterations of all earlier rounds) + t of
# the stream (seed, SETUP, client 0); node = first c whose cumulative share exceeds
# floor(hi32(draw) * sum(shares) / 2^32).  A node may get no iteration in a round: it then
# sends U = 0 at once (Algorithm 3 sends after the inner loop, however short).
def split_mode(cfg) -> int:
    return cfg.get("split_mode", 0)


def client_shares(cfg):
    sh = cfg.get("client_shares")
    return list(sh) if sh else [1] * cfg["n_clients"]


def assign_node(r: int, shares) -> int:
    """Node a coin (one 64-bit draw) falls to."""
    v = ((r >> 32) * sum(shares)) >> 32
    acc = 0
    for c, w in enumerate(shares):
        acc += w
        if v < acc:
            return c
    raise AssertionError("coin outside the shares")


def split_round(cfg, i: int):
    """[s_{i,c} for every node c] of global round i (split_mode 1)."""
    a, b, base = cfg["sched_a"], cfg["sched_b"], cfg["round_base"]
    key = rng.stream_key(cfg["seed"], rng.STREAM_SETUP, 0)
    g0 = samples_before(a, b, base, i)
    shares = client_shares(cfg)
    out = [0] * cfg["n_clients"]
    for t in range(sample_size(a, b, i)):
        out[assign_node(rng.draw(key, g0 + t), shares)] += 1
    return out


def node_sample_size(cfg, c: int, i: int, _cache={}) -> int:
    """s_{i,c}: the node's own sequence (split_mode 0) or its share of the global round (1)."""
    if not split_mode(cfg):
        return sample_size(cfg["sched_a"], cfg["sched_b"], i)
    k = (cfg["seed"], cfg["sched_a"], cfg["sched_b"], cfg["round_base"], cfg["n_clients"],
         tuple(client_shares(cfg)), i)
    if k not in _cache:
        _cache[k] = split_round(cfg, i)
    return _cache[k][c]


def node_samples_before(cfg, c: int, i: int) -> int:
    """Samples node c has consumed before round i."""
    if not split_mode(cfg):
        return samples_before(cfg["sched_a"], cfg["sched_b"], cfg["round_base"], i)
    return sum(node_sample_size(cfg, c, j) for j in range(cfg["round_base"], i))


def new_state(cfg):
    return dict(clock=0, H=[0] * cfg["n_clients"], rounds_done=0)


def _delay(cfg, which, r):
    if cfg["delay_dist"] == 0:
        return rng.exp_ticks(r, rng.to_ticks(cfg[which + "_delay_mean"]))
    return rng.uniform_ticks(r, rng.to_ticks(cfg[which + "_delay_lo"]),
                             rng.to_ticks(cfg[which + "_delay_hi"]))


def simulate(cfg, n_rounds, state=None):
    """Run the event schedule for n_rounds more rounds per client, to quiescence.

    Returns (events ordered by seq, summary, state_after).
    """
    n = cfg["n_clients"]
    a, b, base, B = cfg["sched_a"], cfg["sched_b"], cfg["round_base"], cfg["batch"]
    d = cfg["max_lag_d"]
    seed = cfg["seed"]
    st = new_state(cfg) if state is None else state
    H = list(st["H"])
    t0 = st["clock"]
    first = base + st["rounds_done"]
    last = first + n_rounds
    straggler_q16 = rng.to_q16(cfg["straggler_factor"])

    key_c = [rng.stream_key(seed, rng.STREAM_COMPUTE, c) for c in range(n)]
    key_n = [rng.stream_key(seed, rng.STREAM_NETWORK, c) for c in range(n)]
    ready = [t0] * n
    blocked = {}
    heap = [(t0, START, c, first) for c in range(n)] if n_rounds > 0 else []
    heapq.heapify(heap)
    events = []
    by_task = {}
    seq = 0

    def min_other(c):
        if n == 1:
            return None
        m = min(H)
        if H[c] != m or H.count(m) > 1:
            return m
        return min(H[e] for e in range(n) if e != c)

    def lag_of(c, i):
        m = min_other(c)
        return 0 if m is None else max(0, (i - base) - m)

    while heap:
        t, kind, c, i = heapq.heappop(heap)
        if kind == APPLY:
            H[c] += 1
            by_task[(c, i)]["seq"] = seq
            seq += 1
            for bc in sorted(blocked):
                if d == NEVER_WAIT or lag_of(bc, blocked[bc]) <= d:
                    heapq.heappush(heap, (t, START, bc, blocked.pop(bc)))
            continue
        lag = lag_of(c, i)
        if d != NEVER_WAIT and lag > d:
            blocked[c] = i
            continue
        s = node_sample_size(cfg, c, i)
        if s % B:
            raise ValueError("batch must divide every s_i")
        steps = s // B
        it0 = node_samples_before(cfg, c, i) // B
        straggler = c >= n - cfg["n_stragglers"]
        busy = 0
        for j in range(steps):
            dt = _delay(cfg, "compute", rng.draw(key_c[c], it0 + j))
            if straggler:
                dt = max(1, (dt * straggler_q16) >> 16)
            busy += dt
        t_trigger = t + busy
        t_apply = t_trigger + _delay(cfg, "network", rng.draw(key_n[c], i))
        by_task[(c, i)] = ev = dict(t_start=t, t_trigger=t_trigger, t_apply=t_apply,
                                    wait_ticks=t - ready[c], client=c, round=i, samples=s,
                                    steps=steps, seq=None, seen=seq, lag=lag)
        events.append(ev)
        heapq.heappush(heap, (t_apply, APPLY, c, i))
        ready[c] = t_trigger
        if i + 1 < last:
            heapq.heappush(heap, (t_trigger, START, c, i + 1))

    assert not blocked and all(e["seq"] is not None for e in events)
    events.sort(key=lambda e: e["seq"])
    samples_total = sum(e["samples"] for e in events)
    s_first = sample_size(a, b, base)
    if split_mode(cfg):
        s_first = max(1, s_first // n)     # a node's expected share of the first global round
    per_client = samples_total // n if n else 0
    summary = dict(
        messages_up=len(events), model_pulls=len(events), samples_total=samples_total,
        messages_if_per_sample=samples_total // B,
        messages_if_constant_b=(n * -(-per_client // s_first)) if s_first else 0,
        t_end_ticks=max((e["t_apply"] for e in events), default=t0))
    after = dict(clock=summary["t_end_ticks"], H=H, rounds_done=st["rounds_done"] + n_rounds)
    return events, summary, after


# ---- peer-to-peer ring (Section 1, Fig. 1b; the topology of the paper's experiments) ----
# Every node keeps its own model and history map.  A round's sum (c, U_i, i) goes to the node's
# ring neighbours only (Algorithm 3: "Send a tuple (c, U_i, i) to the other c's neighbors") and is
# not forwarded (Algorithm 3 has no relay step).  Receive bumps H_v[c] when the message arrives;
# Synchronize(H, d, i) looks at the node's neighbours only.  One network delay per message and
# destination: draw number 2 * round + side of the sender's network stream (side 0 = node c - 1,
# side 1 = node c + 1; a node with a single neighbour uses side 0).  Ties: (tick, RECEIVE before
# START, node, then sender and round).  A log record is one delivery (sender, round, destination);
# a node without neighbours logs its rounds with destination NO_DEST.
RECEIVE = 0
NO_DEST = 0xFFFFFFFF


def ring_neighbours(n: int, c: int):
    """Neighbours of node c with the side each one sits on: [(side, node)]."""
    out = []
    for side, v in ((0, (c - 1) % n), (1, (c + 1) % n)):
        if v != c and v not in [w for _, w in out]:
            out.append((side, v))
    return out


def new_ring_state(cfg):
    n = cfg["n_clients"]
    return dict(clock=0, H=[{v: 0 for _, v in ring_neighbours(n, c)} for c in range(n)], rounds_done=0)


def simulate_ring(cfg, n_rounds, state=None):
    """Event schedule of the ring for n_rounds more rounds per node, to quiescence.

    Returns (tasks, deliveries, summary, state_after).  tasks: one dict per round-task in
    (t_trigger, client, round) order with `task` = its position there and `applied` = the
    deliveries (indices into deliveries) that reached the node before the round started and
    after its previous start.  deliveries: one dict per (sender, round, destination) in
    processing order = (t_apply, dest, client, round), `seq` = its position."""
    n = cfg["n_clients"]
    a, b, base, B = cfg["sched_a"], cfg["sched_b"], cfg["round_base"], cfg["batch"]
    d, seed = cfg["max_lag_d"], cfg["seed"]
    st = new_ring_state(cfg) if state is None else state
    H = [dict(h) for h in st["H"]]
    t0 = st["clock"]
    first = base + st["rounds_done"]
    last = first + n_rounds
    straggler_q16 = rng.to_q16(cfg["straggler_factor"])
    key_c = [rng.stream_key(seed, rng.STREAM_COMPUTE, c) for c in range(n)]
    key_n = [rng.stream_key(seed, rng.STREAM_NETWORK, c) for c in range(n)]
    nbrs = [ring_neighbours(n, c) for c in range(n)]
    ready = [t0] * n
    blocked = {}
    pending = [[] for _ in range(n)]          # deliveries that reached a node since its last start
    n_received = [0] * n
    heap = [(t0, START, c, first, 0) for c in range(n)] if n_rounds > 0 else []
    heapq.heapify(heap)
    tasks, deliveries = [], []

    def lag_of(c, i):
        if not H[c]:
            return 0
        return max(0, (i - base) - min(H[c].values()))

    while heap:
        t, kind, node, x, y = heapq.heappop(heap)
        if kind == RECEIVE:
            sender, rnd = x, y
            H[node][sender] += 1
            dl = next(q for q in deliveries if q["seq"] is None and q["dest"] == node and q["client"] == sender
                      and q["round"] == rnd)
            dl["seq"] = sum(1 for q in deliveries if q["seq"] is not None)
            pending[node].append(dl)
            n_received[node] += 1
            if node in blocked and (d == NEVER_WAIT or lag_of(node, blocked[node]) <= d):
                heapq.heappush(heap, (t, START, node, blocked.pop(node), 0))
            continue
        c, i = node, x
        lag = lag_of(c, i)
        if d != NEVER_WAIT and lag > d:
            blocked[c] = i
            continue
        s = node_sample_size(cfg, c, i)
        if s % B:
            raise ValueError("batch must divide every s_i")
        steps = s // B
        it0 = node_samples_before(cfg, c, i) // B
        straggler = c >= n - cfg["n_stragglers"]
        busy = 0
        for j in range(steps):
            dt = _delay(cfg, "compute", rng.draw(key_c[c], it0 + j))
            if straggler:
                dt = max(1, (dt * straggler_q16) >> 16)
            busy += dt
        t_trigger = t + busy
        task = dict(t_start=t, t_trigger=t_trigger, wait_ticks=t - ready[c], client=c, round=i, samples=s,
                    steps=steps, seen=n_received[c], lag=lag, applied=[q for q in pending[c]], task=None)
        pending[c] = []
        tasks.append(task)
        for side, v in nbrs[c]:
            t_arr = t_trigger + _delay(cfg, "network", rng.draw(key_n[c], 2 * i + side))
            deliveries.append(dict(task, t_apply=t_arr, dest=v, seq=None, of_task=task))
            heapq.heappush(heap, (t_arr, RECEIVE, v, c, i))
        if not nbrs[c]:
            deliveries.append(dict(task, t_apply=t_trigger, dest=NO_DEST, seq=None, of_task=task))
        ready[c] = t_trigger
        if i + 1 < last:
            heapq.heappush(heap, (t_trigger, START, c, i + 1, 0))

    assert not blocked
    # a node without neighbours: its records take the places the trigger times give them
    lone = sorted((q for q in deliveries if q["dest"] == NO_DEST), key=lambda q: (q["t_apply"], q["client"], q["round"]))
    for k, q in enumerate(lone):
        q["seq"] = k
    assert all(q["seq"] is not None for q in deliveries)
    deliveries.sort(key=lambda q: q["seq"])
    tasks.sort(key=lambda e: (e["t_trigger"], e["client"], e["round"]))
    for k, e in enumerate(tasks):
        e["task"] = k
    for q in deliveries:
        q["task"] = q["of_task"]["task"]
    samples_total = sum(e["samples"] for e in tasks)
    s_first = sample_size(a, b, base)
    if split_mode(cfg):
        s_first = max(1, s_first // n)
    per_client = samples_total // n if n else 0
    n_links = sum(len(v) for v in nbrs)
    summary = dict(
        messages_up=sum(1 for q in deliveries if q["dest"] != NO_DEST), model_pulls=0, samples_total=samples_total,
        messages_if_per_sample=(samples_total // B) * (n_links // n if n else 0),
        messages_if_constant_b=(n_links * -(-per_client // s_first)) if s_first else 0,
        t_end_ticks=max([q["t_apply"] for q in deliveries] + [t0]))
    after = dict(clock=summary["t_end_ticks"], H=H, rounds_done=st["rounds_done"] + n_rounds)
    return tasks, deliveries, summary, after


def pack_ring_events(deliveries) -> bytes:
    """The ring's log as the library lays it out: one 64-byte record per delivery."""
    out = bytearray()
    for q in deliveries:
        out += EVENT_STRUCT.pack(q["t_start"], q["t_trigger"], q["t_apply"], q["wait_ticks"],
                                 q["client"], q["round"], q["samples"], q["steps"],
                                 q["seq"], q["seen"], q["lag"], q["dest"])
    return bytes(out)


def pack_events(events) -> bytes:
    """The event log as the library lays it out (64 bytes per record)."""
    out = bytearray()
    for e in events:
        out += EVENT_STRUCT.pack(e["t_start"], e["t_trigger"], e["t_apply"], e["wait_ticks"],
                                 e["client"], e["round"], e["samples"], e["steps"],
                                 e["seq"], e["seen"], e["lag"], 0)
    return bytes(out)
