"""The whole hot path, sequentially: every client's local-SGD rounds and the
server's ordered aggregation.

TEST INFRASTRUCTURE (see the package header).  fp64 throughout.

Algorithm 3, MainComputeNode: a round sets h = 0, U_i = 0 and repeats s_{i,c}
times: sample xi from D_c; g = grad f(w_c, xi); w_c -= eta_i * g; U_i += g;
then sends (c, U_i, i).  Receive: w -= eta_k * U.  Section 1 (client-server
form): the server aggregates the received update sums into a global model that
clients pick up.  Reading used here: a message takes effect at the receiver's
next round start, so a client starts round i from the server's model at that
time minus its own update sums that are still in flight (they are already in
its local model through line "w_c -= eta_i g").
"""
import numpy as np

from . import models, rng, schedule


def f32(v) -> float:
    """The library's config carries lr, lr_beta and l2 as fp32; use those values."""
    return float(np.float32(v))


def step_size(cfg, i, c=0):
    """Round step size of node c's round i: t = the node's own iterations before the round
    (every node has the same count unless the Setup split of Algorithm 2 is on)."""
    t = schedule.node_samples_before(cfg, c, i) // cfg["batch"]
    return schedule.round_step_size(f32(cfg["lr"]), f32(cfg["lr_beta"]), t)


def task_indices(cfg, c, i, n_c):
    """Sample indices of round-task (c, i), shape [steps, B] (with replacement,
    keyed by the client's running sample counter)."""
    B = cfg["batch"]
    k0 = schedule.node_samples_before(cfg, c, i)
    s = schedule.node_sample_size(cfg, c, i)
    key = rng.stream_key(cfg["seed"], rng.STREAM_SAMPLE, c)
    idx = [rng.sample_index(rng.draw(key, k0 + k), n_c) for k in range(s)]
    return np.asarray(idx, dtype=np.int64).reshape(s // B, B)


def run_task(cfg, client_data, c, i, w_start):
    """One round of client c from model w_start: returns (U_i, w_end)."""
    X, y = client_data
    dims, l2, prec = cfg["dims"], f32(cfg["l2"]), cfg["precision"]
    eta = step_size(cfg, i, c)
    w = np.array(w_start, dtype=np.float64)
    U = np.zeros_like(w)
    for idx in task_indices(cfg, c, i, len(y)):
        if cfg["model"] == 2:      # the small convolutional classifier
            _, g = models.cnn_loss_and_grad(w, X[idx], y[idx], dims, l2)
        else:
            _, g = models.loss_and_grad(w, X[idx], y[idx], dims, l2, prec)
        w -= eta * g
        U += g
    return U, w


def run(cfg, data, w0, n_rounds=None, keep=False, state=None):
    """All clients, n_rounds rounds each, to quiescence.

    w0 is the server model the call starts from; state (from a previous call's
    result) continues the simulated clock, histories and round counters.
    keep: True keeps every round's start model, a collection of seq numbers only those.
    Returns dict(events, summary, w, U (by seq), w_start (by seq, where kept), state).
    """
    n_rounds = cfg["n_rounds"] if n_rounds is None else n_rounds
    events, summary, state_after = schedule.simulate(cfg, n_rounds, state)
    order = sorted([(e["t_apply"], schedule.APPLY, e["client"], e["round"], e) for e in events] +
                   [(e["t_start"], schedule.START, e["client"], e["round"], e) for e in events],
                   key=lambda r: r[:4])
    w_g = np.array(w0, dtype=np.float64)
    U_by_seq = [None] * len(events)
    w_start_by_seq = [None] * len(events)
    in_flight = {c: [] for c in range(cfg["n_clients"])}
    for _, kind, c, i, e in order:
        if kind == schedule.START:
            w_start = w_g.copy()
            for f in in_flight[c]:
                w_start -= step_size(cfg, f["round"], c) * U_by_seq[f["seq"]]
            U, _ = run_task(cfg, data[c], c, i, w_start)
            U_by_seq[e["seq"]] = U
            if keep is True or (keep and e["seq"] in keep):
                w_start_by_seq[e["seq"]] = w_start
            in_flight[c].append(e)
        else:
            w_g -= step_size(cfg, i, c) * U_by_seq[e["seq"]]
            in_flight[c].remove(e)
    assert all(not v for v in in_flight.values())
    return dict(events=events, summary=summary, w=w_g, U=U_by_seq, w_start=w_start_by_seq,
                state=state_after)


def run_ring(cfg, data, w0, n_rounds=None, keep=False, state=None, node_models=None):
    """The peer-to-peer ring (Section 1, Fig. 1b): every node keeps its own model.

    A node's round starts from its own model after the update sums that reached it since its
    previous start have been applied (Receive: w_c -= eta_k * U, in arrival order); its own sum
    is applied when the round ends (w_c -= eta_i * U_i, the net effect of the inner loop); sums are
    not forwarded.  Returns dict(tasks, deliveries, summary, W (node models at quiescence),
    U (by task), w_start (by task, where kept), state)."""
    n = cfg["n_clients"]
    n_rounds = cfg["n_rounds"] if n_rounds is None else n_rounds
    tasks, deliveries, summary, state_after = schedule.simulate_ring(cfg, n_rounds, state)
    W = [np.array(w0 if node_models is None else node_models[c], dtype=np.float64) for c in range(n)]
    U_by_task = [None] * len(tasks)
    w_start_by_task = [None] * len(tasks)
    applied = set()
    for e in sorted(tasks, key=lambda e: (e["t_start"], e["client"], e["round"])):
        c = e["client"]
        for q in e["applied"]:
            W[c] -= step_size(cfg, q["round"], q["client"]) * U_by_task[q["task"]]
            applied.add(q["seq"])
        w_start = W[c].copy()
        U, _ = run_task(cfg, data[c], c, e["round"], w_start)
        U_by_task[e["task"]] = U
        if keep is True or (keep and e["task"] in keep):
            w_start_by_task[e["task"]] = w_start
        W[c] -= step_size(cfg, e["round"], c) * U
    for q in deliveries:                       # quiescence: what is still on its way arrives
        if q["dest"] != schedule.NO_DEST and q["seq"] not in applied:
            W[q["dest"]] -= step_size(cfg, q["round"], q["client"]) * U_by_task[q["task"]]
    return dict(tasks=tasks, deliveries=deliveries, summary=summary, W=W, U=U_by_task,
                w_start=w_start_by_task, state=state_after)
