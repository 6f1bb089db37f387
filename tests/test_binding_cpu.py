"""Host-side checks of the library that need no GPU: exported symbols, the
integer generator and delay draws, and the schedule against the checker."""
import ctypes
import os
import re

import pytest

from oracle import rng, schedule
from paper_2112_13935_b200 import _lib, api, build, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "aet.h")).read()
    declared = set(re.findall(r"\b(aet_[a-z_0-9]+)\s*\(", header))
    assert declared == set(_lib.PROTOTYPES), declared ^ set(_lib.PROTOTYPES)
    lib = ctypes.CDLL(_lib.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_sizes_match_the_header_layout():
    assert ctypes.sizeof(_lib.AetEvent) == 64
    assert ctypes.sizeof(_lib.AetSummary) == 48
    cfg = api.make_config(workloads.get_config("cfg1"))
    # the library rejects a config whose struct_size it does not recognise
    ev, _ = api.aet_schedule_only(cfg, 1)
    assert len(ev) == 4
    cfg.struct_size += 4
    with pytest.raises(api.AetError) as e:
        api.aet_schedule_only(cfg, 1)
    assert e.value.status == 1


def test_generator_and_delay_draws_agree_with_the_checker():
    for seed, st, c, k in [(0, 0, 0, 0), (0, 1, 3, 17), (12345, 2, 1023, 2 ** 40), (2 ** 63 + 5, 1, 7, 99)]:
        r = api.aet_debug_draw(seed, st, c, k)
        assert r == rng.draw(rng.stream_key(seed, st, c), k)
        for mean in (1, 104858, 1 << 20, 100 << 20):
            assert api.aet_debug_delay_ticks(0, r, mean) == rng.exp_ticks(r, mean)
        assert api.aet_debug_delay_ticks(1, r, 1000, 5000) == rng.uniform_ticks(r, 1000, 5000)
    for r in (0, 1, 2 ** 64 - 1, 2 ** 63):
        assert api.aet_debug_delay_ticks(0, r, 1 << 20) == rng.exp_ticks(r, 1 << 20)


def test_stored_generator_vectors():
    # vectors written by tests/golden/make_golden.py from the checker alone
    path = os.path.join(ROOT, "tests", "golden", "rng_vectors.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 6
    for seed, st, c, k, r, mean, ticks in rows:
        got = api.aet_debug_draw(int(seed), int(st), int(c), int(k))
        assert got == int(r, 16)
        assert api.aet_debug_delay_ticks(0, got, int(mean)) == int(ticks)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4"])
def test_schedule_is_bit_identical_to_the_checker(name):
    cfg = workloads.get_config(name)
    blob, summary = api.aet_schedule_only(cfg, cfg["n_rounds"], raw=True)
    events, want, _ = schedule.simulate(cfg, cfg["n_rounds"])
    assert blob == schedule.pack_events(events)
    assert summary == want


@pytest.mark.parametrize("over", [
    dict(max_lag_d=0), dict(max_lag_d=workloads.NEVER_WAIT), dict(n_clients=1),
    dict(delay_dist=1), dict(n_stragglers=3, straggler_factor=37.5, max_lag_d=2),
    dict(round_base=1, sched_b=0, lr_beta=0.01), dict(network_delay_mean=50.0, n_clients=9, max_lag_d=3),
    # constant, equal delays: every START coincides with APPLYs (tie rule) and with other STARTs
    dict(n_clients=3, sched_a=0, sched_b=1, delay_dist=1, compute_delay_lo=5 / 2 ** 20, compute_delay_hi=5 / 2 ** 20,
         network_delay_lo=5 / 2 ** 20, network_delay_hi=5 / 2 ** 20, max_lag_d=workloads.NEVER_WAIT),
    dict(n_clients=3, sched_a=0, sched_b=2, delay_dist=1, compute_delay_lo=4 / 2 ** 20, compute_delay_hi=4 / 2 ** 20,
         network_delay_lo=8 / 2 ** 20, network_delay_hi=8 / 2 ** 20, max_lag_d=1),
    # Algorithm 2, Setup: the global round size split among the nodes by coin flips (some rounds are empty)
    dict(split_mode=1, n_clients=5, sched_a=6, sched_b=2),
    dict(split_mode=1, n_clients=3, sched_a=10, sched_b=5, client_shares=[1, 2, 5], lr_beta=0.02, max_lag_d=2),
    dict(split_mode=1, n_clients=1, sched_a=3, sched_b=1),
    dict(split_mode=1, n_clients=12, sched_a=1, sched_b=1, max_lag_d=0),
])
def test_schedule_variants_match_the_checker(over):
    cfg = workloads.get_config("cfg1", **over)
    blob, summary = api.aet_schedule_only(cfg, 7, raw=True)
    events, want, _ = schedule.simulate(cfg, 7)
    assert blob == schedule.pack_events(events) and summary == want


def test_schedule_rejects_bad_configs():
    for over, status in [(dict(batch=3), 2), (dict(n_clients=0), 2), (dict(precision=5), 2),
                         (dict(n_stragglers=9), 2), (dict(lr=0.0), 2), (dict(sched_b=0), 2),
                         (dict(split_mode=2), 2), (dict(split_mode=1, client_shares=[0, 0, 0, 0]), 2),
                         (dict(split_mode=1, model=1, dims=[784, 16, 10], batch=2, sched_a=2, sched_b=2), 2)]:
        with pytest.raises(api.AetError) as e:
            api.aet_schedule_only(workloads.get_config("cfg1", **over), 3)
        assert e.value.status == status, over


def test_wave_plan_counts():
    # one client: every round depends on the previous one
    assert api.aet_debug_plan_waves(workloads.get_config("cfg1", n_clients=1), 5) == 5
    # d = 0: rounds are lock-step, one wave per round
    assert api.aet_debug_plan_waves(workloads.get_config("cfg1", max_lag_d=0), 5) == 5
    w = api.aet_debug_plan_waves(workloads.get_config("cfg2"), 30)
    assert 30 <= w <= 60


def test_create_without_a_gpu_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(api.AetError) as e:
        api.aet_create(workloads.get_config("cfg1"))
    assert e.value.status == 5


def _replay_plan(cfg, n_rounds, events, lay):
    """Walk the launch order (round kernel of wave 0, aggregation 0, wave 1, ...) keeping track of
    what every update-sum row and snapshot slot holds, and check that every read finds what it
    needs: a task its start snapshot and its own sums still in flight, the server every sum it
    applies."""
    E = len(events)
    row_holds = {}            # row -> seq whose update sum it holds
    slot_holds = {0: 0}       # slot -> start position (number of updates applied) it holds
    mine = {}
    for e in events:
        mine.setdefault(e["client"], []).append(e)
    lo, q = 0, 0
    for L in range(lay["waves"]):
        wave = []
        while q < E and lay["task_wave"][q] == L:
            wave.append(q)
            q += 1
        assert wave, "empty wave"
        for t in wave:                                        # reads of the round kernel
            e = events[int(lay["task_seq"][t])]
            assert slot_holds.get(int(lay["task_snap_slot"][t])) == e["seen"], (L, e)
            for f in mine[e["client"]]:
                if f["round"] < e["round"] and f["seq"] >= e["seen"]:
                    assert row_holds.get(int(lay["u_row"][f["seq"]])) == f["seq"], (L, e, f)
        rows = [int(lay["u_row"][int(lay["task_seq"][t])]) for t in wave]
        assert len(set(rows)) == len(rows), "two tasks of a wave share a row"
        for t in wave:                                        # its writes
            row_holds[int(lay["u_row"][int(lay["task_seq"][t])])] = int(lay["task_seq"][t])
        hi = int(lay["apply_upto"][L])
        for k in range(lo, hi):                               # the aggregation, in seq order
            assert row_holds.get(int(lay["u_row"][k])) == k, (L, k)
            s = int(lay["snap_slot_after"][k])
            if s >= 0:
                slot_holds[s] = k + 1
        lo = hi
    assert q == E and lo == E
    assert max(row_holds) < lay["n_u_rows"] and max(slot_holds) < lay["n_snap"]


@pytest.mark.parametrize("name,over", [
    ("cfg1", {}), ("cfg2", {}), ("cfg5", dict(n_clients=128)),
    ("cfg1", dict(n_clients=3, n_rounds=8, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=500.0)),
    ("cfg1", dict(n_clients=7, n_rounds=9, max_lag_d=0)),
    ("cfg2", dict(max_lag_d=3, network_delay_mean=20.0)),
    ("cfg1", dict(split_mode=1, n_clients=9, sched_a=4, sched_b=2, n_rounds=8)),
])
def test_recycled_rows_and_slots_always_hold_what_is_read(name, over):
    cfg = workloads.get_config(name, **over)
    R = cfg["n_rounds"]
    events, _, _ = schedule.simulate(cfg, R)
    lay = api.aet_debug_plan_layout(cfg, R)
    _replay_plan(cfg, R, events, lay)
    keep = api.aet_debug_plan_layout(dict(cfg, flags=api.FLAG_KEEP_UPDATE_SUMS), R)
    _replay_plan(cfg, R, events, keep)
    assert keep["n_u_rows"] == len(events) and list(keep["u_row"]) == list(range(len(events)))
    assert lay["n_u_rows"] <= keep["n_u_rows"] and lay["n_snap"] <= keep["n_snap"]
    assert lay["waves"] == keep["waves"] == api.aet_debug_plan_waves(cfg, R)
    if name == "cfg2" and not over:
        assert lay["n_u_rows"] < len(events) // 4     # recycling pays: rows ~ rounds in flight


@pytest.mark.parametrize("over", [
    dict(n_clients=5), dict(n_clients=5, max_lag_d=0), dict(n_clients=5, max_lag_d=2), dict(n_clients=8, max_lag_d=5),
    dict(n_clients=1), dict(n_clients=2), dict(n_clients=3, network_delay_mean=30.0),
    dict(n_clients=6, n_stragglers=2, straggler_factor=25.0, max_lag_d=1),
    dict(n_clients=7, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=40.0),
    dict(n_clients=5, delay_dist=1, round_base=1, sched_b=0, lr_beta=0.01),              # the paper's own ring setting
    dict(n_clients=4, split_mode=1, sched_a=9, sched_b=4, client_shares=[3, 1, 1, 2]),    # with the Setup split
    # constant, equal delays: many simultaneous arrivals (tie rule: by destination, then sender)
    dict(n_clients=4, sched_a=0, sched_b=1, delay_dist=1, compute_delay_lo=10 / 2 ** 20, compute_delay_hi=10 / 2 ** 20,
         network_delay_lo=25 / 2 ** 20, network_delay_hi=25 / 2 ** 20, max_lag_d=1),
])
def test_ring_schedule_is_bit_identical_to_the_checker(over):
    cfg = workloads.get_config("cfg1", topology=1, **over)
    blob, summary = api.aet_schedule_only(cfg, 7, raw=True)
    tasks, deliveries, want, _ = schedule.simulate_ring(cfg, 7)
    assert blob == schedule.pack_ring_events(deliveries)
    assert summary == want
