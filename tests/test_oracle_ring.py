"""Pins for the checker's peer-to-peer ring (Section 1, Fig. 1b; Algorithm 3 read per node):
special cases that reduce to the client-server form already pinned, the model invariant, the
prose statements about d, and a four-node timeline worked by hand."""
import numpy as np
import pytest

from oracle import schedule, sim
from paper_2112_13935_b200 import workloads

T = 1 << 20   # ticks per time unit


def _const_delays(compute, network, **kw):
    # delay_dist 1 with lo = hi: every SGD iteration takes `compute` ticks, every message `network`
    return dict(delay_dist=1, compute_delay_lo=compute / T, compute_delay_hi=compute / T,
                network_delay_lo=network / T, network_delay_hi=network / T, **kw)


def _cfg(**kw):
    base = dict(topology=1, l2=0.0, n_rounds=4, data=dict(per_client=120))
    base.update(kw)
    return workloads.get_config("cfg1", **base)


def test_ring_neighbours():
    assert schedule.ring_neighbours(1, 0) == []
    assert schedule.ring_neighbours(2, 0) == [(0, 1)] and schedule.ring_neighbours(2, 1) == [(0, 0)]
    assert schedule.ring_neighbours(3, 0) == [(0, 2), (1, 1)]
    assert schedule.ring_neighbours(6, 5) == [(0, 4), (1, 0)]


def test_one_node_ring_is_the_one_client_run():
    # no neighbours: nothing is ever received; the client-server form with one client is pinned to plain SGD
    cfg = _cfg(n_clients=1, n_rounds=5)
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    ring = sim.run_ring(cfg, data, w0)
    star = sim.run(dict(cfg, topology=0), data, w0)
    assert np.abs(ring["W"][0] - star["w"]).max() < 1e-13
    assert ring["summary"]["messages_up"] == 0 and len(ring["deliveries"]) == 5
    assert all(q["dest"] == schedule.NO_DEST and q["t_apply"] == q["t_trigger"] for q in ring["deliveries"])


@pytest.mark.parametrize("n", [2, 3])
def test_small_rings_are_complete_graphs_and_match_the_server_form(n):
    # with 2 or 3 nodes every node neighbours every other one; with constant delays a message reaches a peer
    # exactly when the server of the client-server form would have applied it
    cfg = _cfg(n_clients=n, **_const_delays(3, 7))
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    ring = sim.run_ring(cfg, data, w0, keep=True)
    star = sim.run(dict(cfg, topology=0), data, w0, keep=True)
    for c in range(n):
        assert np.abs(ring["W"][c] - star["w"]).max() < 1e-12
    # and every round started from the same model in both forms
    by_task = {(e["client"], e["round"]): e["task"] for e in ring["tasks"]}
    for e in star["events"]:
        k = by_task[(e["client"], e["round"])]
        assert np.abs(ring["w_start"][k] - star["w_start"][e["seq"]]).max() < 1e-12
        assert ring["tasks"][k]["t_start"] == e["t_start"] and ring["tasks"][k]["t_trigger"] == e["t_trigger"]


def test_node_model_is_w0_minus_own_and_neighbours_sums():
    # Receive applies what the two neighbours sent and nothing is forwarded:
    # w_c = w_0 - sum over e in {c-1, c, c+1} and rounds i of eta_i U_{e,i}
    cfg = _cfg(n_clients=6, n_rounds=5, lr_beta=0.03, n_stragglers=1, straggler_factor=5.0)
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    r = sim.run_ring(cfg, data, w0)
    for c in range(6):
        acc = w0.astype(np.float64)
        for e in r["tasks"]:
            if e["client"] in {(c - 1) % 6, c, (c + 1) % 6}:
                acc -= sim.step_size(cfg, e["round"], e["client"]) * r["U"][e["task"]]
        assert np.abs(acc - r["W"][c]).max() < 1e-12
    assert np.abs(r["W"][0] - r["W"][3]).max() > 1e-3       # nodes three hops apart do differ
    assert r["summary"]["messages_up"] == 6 * 5 * 2


def test_d0_a_node_waits_for_both_neighbours_previous_round():
    # Appendix (asynchronous round d = 0): the nodes wait for each other - here: for their neighbours
    cfg = _cfg(n_clients=7, n_rounds=6, max_lag_d=0, n_stragglers=1, straggler_factor=20.0)
    tasks, deliveries, _, _ = schedule.simulate_ring(cfg, 6)
    arrival = {(q["client"], q["round"], q["dest"]): q["t_apply"] for q in deliveries}
    for e in tasks:
        assert e["lag"] == 0
        if e["round"] > 0:
            for v in ((e["client"] - 1) % 7, (e["client"] + 1) % 7):
                assert arrival[(v, e["round"] - 1, e["client"])] <= e["t_start"]
    assert any(e["wait_ticks"] > 0 for e in tasks)


def test_d1_a_node_runs_at_most_one_round_ahead_of_its_neighbours():
    cfg = _cfg(n_clients=5, n_rounds=8, max_lag_d=1, n_stragglers=1, straggler_factor=100.0)
    tasks, deliveries, _, _ = schedule.simulate_ring(cfg, 8)
    assert max(e["lag"] for e in tasks) == 1
    # the straggler's neighbours wait; the nodes two hops away wait for THEM in turn
    assert all(any(e["wait_ticks"] > 0 for e in tasks if e["client"] == c) for c in (3, 0, 2, 1))
    never = schedule.simulate_ring(dict(cfg, max_lag_d=schedule.NEVER_WAIT), 8)[0]
    assert all(e["wait_ticks"] == 0 for e in never) and max(e["lag"] for e in never) > 1


def test_four_node_timeline_worked_by_hand():
    # 4 nodes, one sample per round (s_i = 1), every iteration 10 ticks, every message 25 ticks, d = 1, 3 rounds.
    # All nodes are alike, so all start round 0 at 0, trigger at 10, and their messages arrive at 35.
    # Round 1 (rel 1): lag = 1 - H = 1 <= d: starts at 10 without waiting, triggers at 20, arrives 45.
    # Round 2 (rel 2) is ready at 20: lag = 2 - 0 = 2 > d: blocked until both neighbours' round-0 messages are in
    # (tick 35; the first of the two arrivals leaves the other neighbour's count at 0), then lag = 2 - 1 = 1:
    # starts at 35 having waited 15, triggers at 45, arrives at 70.
    cfg = _cfg(n_clients=4, n_rounds=3, sched_a=0, sched_b=1, max_lag_d=1, **_const_delays(10, 25))
    tasks, deliveries, summary, after = schedule.simulate_ring(cfg, 3)
    want = {0: (0, 10, 0, 0, 0), 1: (10, 20, 0, 1, 0), 2: (35, 45, 15, 1, 2)}   # round: start, trigger, wait, lag, seen
    for e in tasks:
        assert (e["t_start"], e["t_trigger"], e["wait_ticks"], e["lag"], e["seen"]) == want[e["round"]], e
    assert len(deliveries) == 24 and summary["messages_up"] == 24 and summary["t_end_ticks"] == 70
    assert [q["t_apply"] for q in deliveries] == [35] * 8 + [45] * 8 + [70] * 8
    # order of equal arrival times: by destination, then sender
    assert [(q["dest"], q["client"]) for q in deliveries[:8]] == [(0, 1), (0, 3), (1, 0), (1, 2), (2, 1), (2, 3), (3, 0), (3, 2)]
    assert [q["seq"] for q in deliveries] == list(range(24))
    assert after["H"] == [{3: 3, 1: 3}, {0: 3, 2: 3}, {1: 3, 3: 3}, {2: 3, 0: 3}]
    # round 2 started from a model that holds both neighbours' round-0 sums and not yet their round-1 sums
    r2 = [e for e in tasks if e["round"] == 2 and e["client"] == 0][0]
    assert sorted((q["client"], q["round"]) for q in r2["applied"]) == [(1, 0), (3, 0)]
    # the communication-cost pair: one message per SGD iteration and link instead would be 4 * 3 * 2 as well here
    assert summary["messages_if_per_sample"] == 24


def test_ring_log_is_internally_consistent_and_packs_to_64_bytes():
    cfg = _cfg(n_clients=5, n_rounds=6, network_delay_mean=3.0)
    tasks, deliveries, summary, _ = schedule.simulate_ring(cfg, 6)
    keys = [(q["t_apply"], q["dest"], q["client"], q["round"]) for q in deliveries]
    assert keys == sorted(keys)
    assert len(schedule.pack_ring_events(deliveries)) == 64 * len(deliveries)
    for e in tasks:
        mine = [q for q in deliveries if q["dest"] == e["client"] and q["t_apply"] <= e["t_start"]]
        assert e["seen"] == len(mine)
        assert e["t_start"] <= e["t_trigger"]
    assert [e["task"] for e in tasks] == list(range(len(tasks)))
    assert summary["samples_total"] == 5 * sum(10 * i + 10 for i in range(6))
