"""Pins for the checker's schedule: the paper's printed round counts, closed
forms, the prose special cases for d, and a two-client timeline worked by hand."""
import math
import os

import pytest

from oracle import rng, schedule
from paper_2112_13935_b200 import workloads

HERE = os.path.dirname(os.path.abspath(__file__))


def _paper_rows():
    rows = []
    with open(os.path.join(HERE, "golden", "paper_round_counts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                kind, K, a, b, base, rounds = line.split()
                rows.append((kind, int(K), int(a), int(b), int(base), int(rounds)))
    return rows


@pytest.mark.parametrize("row", _paper_rows())
def test_round_counts_printed_in_the_paper(row):
    _, K, a, b, base, rounds = row
    assert schedule.rounds_needed(K, a, b, base) == rounds


def test_rounds_grow_like_sqrt_K():
    # Section 4.1: T is proportional to sqrt(K) for a linear sequence.
    for K in (10_000, 60_000, 1_000_000):
        T = schedule.rounds_needed(K, 10, 0, 1)
        assert abs(T - math.sqrt(2 * K / 10)) <= 1.0


@pytest.mark.parametrize("name,per_client,total,events", [
    ("cfg1", 150, 600, 20), ("cfg2", 9300, 148800, 480), ("cfg3", 52480, 1679360, 1280),
    ("cfg4", 59520, 3809280, 1920), ("cfg5", 440, 450560, 10240)])
def test_sample_totals_closed_form(name, per_client, total, events):
    cfg = workloads.get_config(name)
    a, b, R = cfg["sched_a"], cfg["sched_b"], cfg["n_rounds"]
    assert a * R * (R - 1) // 2 + b * R == per_client
    assert schedule.samples_before(a, b, 0, R) == per_client
    assert per_client * cfg["n_clients"] == total
    assert cfg["n_clients"] * R == events


def test_round_step_size_values_worked_by_hand():
    # Section 4.1: eta_t = eta_0 / (1 + beta sqrt(t)); Appendix Table 2: eta_0 = 0.01, beta = 0.01.
    # t = 10,000: sqrt = 100, 1 + 0.01 * 100 = 2, so the step is eta_0 / 2; t = 0: eta_0 itself;
    # t = 2,500: sqrt = 50, 1 + 0.5 = 1.5; beta = 0 keeps the step constant.
    assert schedule.round_step_size(0.01, 0.01, 10_000) == 0.005
    assert schedule.round_step_size(0.01, 0.01, 0) == 0.01
    assert abs(schedule.round_step_size(0.01, 0.01, 2_500) - 0.01 / 1.5) < 1e-18
    assert schedule.round_step_size(0.3, 0.0, 123_456) == 0.3
    # as the simulator uses it: t = the client's own iterations before the round.  Paper's schedule
    # s_i = 10 i from round 1, batch 1: before round 5 a client has done 10 + 20 + 30 + 40 = 100
    # iterations, so eta = 0.01 / (1 + 0.01 * 10) = 0.01 / 1.1
    from oracle import sim
    cfg = dict(sched_a=10, sched_b=0, round_base=1, batch=1, lr=0.01, lr_beta=0.01)
    lr32, beta32 = sim.f32(0.01), sim.f32(0.01)
    assert abs(sim.step_size(cfg, 5) - lr32 / (1.0 + beta32 * 10.0)) < 1e-18
    assert sim.step_size(cfg, 1) == lr32


def _check_log(cfg, events, summary):
    n, R = cfg["n_clients"], len(events) // cfg["n_clients"]
    assert [e["seq"] for e in events] == list(range(len(events)))
    keys = [(e["t_apply"], e["client"], e["round"]) for e in events]
    assert keys == sorted(keys)
    for e in events:
        assert e["t_start"] <= e["t_trigger"] < e["t_apply"]
        assert e["samples"] == cfg["sched_a"] * e["round"] + cfg["sched_b"]
        assert e["steps"] * cfg["batch"] == e["samples"]
        assert e["seen"] == sum(1 for f in events if f["t_apply"] <= e["t_start"])
        if cfg["max_lag_d"] != schedule.NEVER_WAIT:
            assert e["lag"] <= cfg["max_lag_d"]
    by = {(e["client"], e["round"]): e for e in events}
    for (c, i), e in by.items():
        if (c, i - 1) in by:
            ready = by[(c, i - 1)]["t_trigger"]
            assert e["t_start"] == ready + e["wait_ticks"]
    assert summary["messages_up"] == n * R == summary["model_pulls"]
    assert summary["samples_total"] == sum(e["samples"] for e in events)
    assert summary["t_end_ticks"] == events[-1]["t_apply"]


def test_log_is_internally_consistent_cfg1_and_cfg2():
    for name in ("cfg1", "cfg2"):
        cfg = workloads.get_config(name)
        events, summary, _ = schedule.simulate(cfg, cfg["n_rounds"])
        _check_log(cfg, events, summary)
        assert summary["samples_total"] == {"cfg1": 600, "cfg2": 148800}[name]


def test_d0_every_client_waits_for_all_previous_rounds():
    # Appendix: with d = 0 "all the compute nodes need to wait for each other".
    cfg = workloads.get_config("cfg1", max_lag_d=0, n_clients=5, n_rounds=6)
    events, _, _ = schedule.simulate(cfg, 6)
    for e in events:
        prev = [f for f in events if f["round"] == e["round"] - 1 and f["client"] != e["client"]]
        assert all(f["t_apply"] <= e["t_start"] for f in prev)


def test_d1_at_most_one_round_ahead_and_fast_clients_wait_for_a_straggler():
    # Appendix: d = 1 lets a node run at most one round ahead of its neighbours.
    cfg = workloads.get_config("cfg1", n_clients=4, n_rounds=8, n_stragglers=1, straggler_factor=100.0)
    events, _, _ = schedule.simulate(cfg, 8)
    assert max(e["lag"] for e in events) <= 1
    fast_wait = sum(e["wait_ticks"] for e in events if e["client"] < 3)
    assert fast_wait > 0
    free = workloads.get_config("cfg1", n_clients=4, n_rounds=8, n_stragglers=1,
                                straggler_factor=100.0, max_lag_d=schedule.NEVER_WAIT)
    ev2, _, _ = schedule.simulate(free, 8)
    assert all(e["wait_ticks"] == 0 for e in ev2)
    assert max(e["lag"] for e in ev2) > 1


def test_single_client_never_waits():
    cfg = workloads.get_config("cfg1", n_clients=1, max_lag_d=0)
    events, _, _ = schedule.simulate(cfg, 5)
    assert all(e["wait_ticks"] == 0 and e["lag"] == 0 for e in events)
    # one client, in-order starts: round i starts when round i-1 triggered
    by = sorted(events, key=lambda e: e["round"])
    for p, q in zip(by, by[1:]):
        assert q["t_start"] == p["t_trigger"]


def hand_cfg():
    """Two clients, three rounds, s_i = i + 1, constant delays: 4 ticks per
    iteration (client 1: x3 = 12), 5 ticks per message, d = 1."""
    tick = 1.0 / (1 << 20)
    return workloads.get_config(
        "cfg1", n_clients=2, n_rounds=3, sched_a=1, sched_b=1, delay_dist=1,
        compute_delay_lo=4 * tick, compute_delay_hi=4 * tick,
        network_delay_lo=5 * tick, network_delay_hi=5 * tick,
        n_stragglers=1, straggler_factor=3.0, max_lag_d=1)


# (client, round): t_start, t_trigger, t_apply, wait, seq, seen, lag -- worked by hand:
#  t=0   both start round 0.                c0: 0->4->9      c1: 0->12->17
#  t=4   c0 starts round 1 (H_1=0, lag 1).  c0: 4->12->17
#  t=9   APPLY (0,0) seq 0.
#  t=12  c0 wants round 2: lag 2 > 1, blocked.  c1 starts round 1 (seen 1): 12->36->41
#  t=17  APPLY (0,1) seq 1, APPLY (1,0) seq 2 (tie: client order); c0 released:
#        round 2 starts at 17 (seen 3, waited 5, lag 1): 17->29->34
#  t=34  APPLY (0,2) seq 3.
#  t=36  c1 starts round 2 (seen 4, lag 0): 36->72->77
#  t=41  APPLY (1,1) seq 4.   t=77  APPLY (1,2) seq 5.
HAND = {
    (0, 0): (0, 4, 9, 0, 0, 0, 0), (1, 0): (0, 12, 17, 0, 2, 0, 0),
    (0, 1): (4, 12, 17, 0, 1, 0, 1), (1, 1): (12, 36, 41, 0, 4, 1, 0),
    (0, 2): (17, 29, 34, 5, 3, 3, 1), (1, 2): (36, 72, 77, 0, 5, 4, 0),
}


def test_two_client_timeline_worked_by_hand():
    cfg = hand_cfg()
    events, summary, _ = schedule.simulate(cfg, 3)
    got = {(e["client"], e["round"]): (e["t_start"], e["t_trigger"], e["t_apply"], e["wait_ticks"],
                                       e["seq"], e["seen"], e["lag"]) for e in events}
    assert got == HAND
    assert summary["t_end_ticks"] == 77 and summary["samples_total"] == 12
    assert summary["messages_if_per_sample"] == 12 and summary["messages_if_constant_b"] == 12


def test_apply_precedes_start_on_equal_ticks():
    # Two equal clients, one sample per round, 5 ticks per iteration and per message, no waiting:
    # rounds start at 0, 5, 10, ...; the updates of round i arrive at 5 i + 10, exactly when
    # round i + 2 starts.  By the tie rule the server applies them first, so round i + 2 sees them.
    tick = 1.0 / (1 << 20)
    cfg = workloads.get_config("cfg1", n_clients=2, sched_a=0, sched_b=1, delay_dist=1,
                               compute_delay_lo=5 * tick, compute_delay_hi=5 * tick,
                               network_delay_lo=5 * tick, network_delay_hi=5 * tick,
                               max_lag_d=schedule.NEVER_WAIT)
    events, _, _ = schedule.simulate(cfg, 4)
    for e in events:
        assert (e["t_start"], e["t_trigger"], e["t_apply"]) == (5 * e["round"], 5 * e["round"] + 5, 5 * e["round"] + 10)
        assert e["seen"] == 2 * max(0, e["round"] - 1)
        assert e["seq"] == 2 * e["round"] + e["client"]


def test_communication_cost_ratio_of_the_papers_setting():
    # K = 60,000 per node with s_i = 10 i from round 1: 110 messages per node
    # against 60,000 (one per sample) and 6,000 (constant s = 10, Table 5).
    cfg = workloads.get_config("cfg1", n_clients=2, sched_a=10, sched_b=0, round_base=1,
                               delay_dist=1, compute_delay_lo=2e-6, compute_delay_hi=2e-6)
    _, summary, _ = schedule.simulate(cfg, 110)
    per_node = summary["samples_total"] // 2
    assert per_node == 61050 and per_node - 10 * 110 < 60000 <= per_node
    assert summary["messages_up"] == 2 * 110
    assert summary["messages_if_per_sample"] == 2 * per_node
    assert summary["messages_if_constant_b"] == 2 * math.ceil(per_node / 10)


def test_run_can_be_continued():
    cfg = workloads.get_config("cfg1")
    ev_a, _, st = schedule.simulate(cfg, 2)
    ev_b, _, st2 = schedule.simulate(cfg, 3, st)
    assert st2["rounds_done"] == 5 and st2["H"] == [5] * 4
    assert min(e["t_start"] for e in ev_b) == st["clock"] == max(e["t_apply"] for e in ev_a)
    assert {e["round"] for e in ev_b} == {2, 3, 4}


def test_packed_log_layout():
    cfg = hand_cfg()
    events, _, _ = schedule.simulate(cfg, 3)
    blob = schedule.pack_events(events)
    assert len(blob) == 64 * 6
    first = schedule.EVENT_STRUCT.unpack_from(blob, 0)
    assert first == (0, 4, 9, 0, 0, 0, 1, 1, 0, 0, 0, 0)


# ---- Algorithm 2 "Setup": the coin-flip split of the global round size ----
def _split_cfg(**kw):
    return workloads.get_config("cfg1", split_mode=1, l2=0.0, **kw)


def test_setup_split_conserves_every_round_and_reduces_to_one_node():
    # s_{i,c} = |{t : a(i,t) = c}|: every iteration of a round goes to exactly one node
    cfg = _split_cfg(n_clients=7, sched_a=10, sched_b=3)
    for i in range(12):
        per_node = schedule.split_round(cfg, i)
        assert sum(per_node) == 10 * i + 3 and len(per_node) == 7 and min(per_node) >= 0
        assert per_node == [schedule.node_sample_size(cfg, c, i) for c in range(7)]
    one = _split_cfg(n_clients=1, sched_a=10, sched_b=3)
    assert [schedule.node_sample_size(one, 0, i) for i in range(6)] == [10 * i + 3 for i in range(6)]
    assert schedule.node_samples_before(one, 0, 4) == 3 + 13 + 23 + 33


def test_setup_split_expectation_is_p_c_times_s_i():
    # E[s_{i,c}] = p_c s_i (the remark after Algorithm 2); shares 1 : 3 : 4 over 8,000 coins
    cfg = _split_cfg(n_clients=3, sched_a=0, sched_b=8000, client_shares=[1, 3, 4])
    got = schedule.split_round(cfg, 0)
    for c, p in enumerate((1 / 8, 3 / 8, 4 / 8)):
        sd = (8000 * p * (1 - p)) ** 0.5
        assert abs(got[c] - 8000 * p) < 4.5 * sd, (c, got)
    # equal shares: p_c = 1/n, chi-square over 5 nodes (4 degrees of freedom, 0.999 quantile 18.5)
    uni = schedule.split_round(_split_cfg(n_clients=5, sched_a=0, sched_b=10000), 0)
    assert sum((g - 2000) ** 2 / 2000 for g in uni) < 18.5


def test_setup_split_uses_a_fresh_coin_for_every_iteration_of_every_round():
    # rounds do not repeat one another's coins, and a round's split does not depend on how far the run goes
    cfg = _split_cfg(n_clients=4, sched_a=0, sched_b=64)
    rounds = [schedule.split_round(cfg, i) for i in range(6)]
    assert len({tuple(r) for r in rounds}) > 1
    seq = []
    key = rng.stream_key(cfg["seed"], rng.STREAM_SETUP, 0)
    for g in range(6 * 64):
        seq.append(schedule.assign_node(rng.draw(key, g), [1, 1, 1, 1]))
    assert len(set(zip(seq[:64], seq[64:128]))) > 4          # consecutive rounds are not copies of each other
    for i in range(6):
        assert rounds[i] == [seq[64 * i:64 * i + 64].count(c) for c in range(4)]
    # assign_node on the extremes of the coin: first and last node
    assert schedule.assign_node(0, [2, 1, 1]) == 0 and schedule.assign_node((1 << 64) - 1, [2, 1, 1]) == 2
    assert schedule.assign_node(1 << 63, [2, 1, 1]) == 1      # v = floor(2^31 * 4 / 2^32) = 2: past node 0's two shares


def test_setup_split_log_counts_and_step_sizes_follow_each_nodes_own_sequence():
    from oracle import sim
    cfg = _split_cfg(n_clients=3, sched_a=6, sched_b=3, n_rounds=6, lr_beta=0.05, client_shares=[1, 2, 3])
    events, summary, _ = schedule.simulate(cfg, 6)
    assert len(events) == 18 and summary["samples_total"] == sum(6 * i + 3 for i in range(6))
    for e in events:
        assert e["samples"] == schedule.node_sample_size(cfg, e["client"], e["round"]) == e["steps"]
        assert e["t_start"] <= e["t_trigger"] < e["t_apply"]
        if e["samples"] == 0:
            assert e["t_trigger"] == e["t_start"]             # nothing to compute: the (zero) sum goes out at once
    # node 2 runs about three times node 0's iterations, so its step size has diminished further by round 5
    assert schedule.node_samples_before(cfg, 2, 5) > schedule.node_samples_before(cfg, 0, 5)
    assert sim.step_size(cfg, 5, 2) < sim.step_size(cfg, 5, 0) < sim.f32(cfg["lr"])
    t0 = schedule.node_samples_before(cfg, 0, 5)
    assert abs(sim.step_size(cfg, 5, 0) - sim.f32(cfg["lr"]) / (1 + sim.f32(0.05) * t0 ** 0.5)) < 1e-15
