"""GPU parity of the softmax-regression path against the CPU checker."""
import numpy as np
import pytest
import torch

from oracle import models, schedule, sim
from paper_2112_13935_b200 import api, workloads
from gpu_helpers import (LOSS_TOL, U_TOL, check_against_oracle, check_round_U, make, rel_err,
                         run_gpu, to_device)

pytestmark = pytest.mark.gpu


def test_cfg1_every_round_U_from_the_checkers_start_model():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0, keep=True)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        worst = max(check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["seq"]])
                    for e in ref["events"])
    assert worst <= U_TOL


def test_cfg1_end_to_end():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    for k, u in enumerate(gpu["U"]):
        assert rel_err(u, ref["U"][k]) <= 1e-4, k     # start models differ by fp32 round-off here
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5
    assert gpu["stats"]["launches"][0] == gpu["stats"]["waves"] == api.aet_debug_plan_waves(cfg, 5)


def test_cfg2_end_to_end_full_size():
    cfg = workloads.get_config("cfg2")
    data, w0 = make(cfg)
    assert sorted(len(y) for _, y in data)[0] >= 8 and sum(len(y) for _, y in data) == 60000
    ref = sim.run(cfg, data, w0, keep=True)
    gpu = run_gpu(cfg, data, w0)
    f_gpu, f_ref = check_against_oracle(cfg, data, w0, gpu, ref)
    assert f_ref < np.log(10.0)                        # it trained (hot: 16 summed clients)
    # invariant at any size: w_g = w_0 - sum eta_k U_k over the GPU's own update sums
    acc = w0.astype(np.float64)
    for e in ref["events"]:
        acc -= sim.step_size(cfg, e["round"]) * gpu["U"][e["seq"]].astype(np.float64)
    assert np.abs(acc - gpu["w"]).max() <= 2e-6 * max(1.0, np.abs(acc).max())
    # sampled round-tasks restarted from the checker's model
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for k in (0, 17, 200, 333, 479):
            e = ref["events"][k]
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][k])


def test_cfg5_shape_64_clients_end_to_end():
    cfg = workloads.get_config("cfg5", n_clients=64)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    gpu = run_gpu(cfg, data, w0, want_U=False)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 2e-5


def test_cfg5_full_size_against_the_checker():
    # 1,024 clients: the configuration the roofline figure is quoted on (waves of up to 1,024 round-tasks)
    cfg = workloads.get_config("cfg5")
    data, w0 = make(cfg)
    sampled = {0: None, 1023: None, 4000: None, 7777: None, 10239: None}
    ref = sim.run(cfg, data, w0, keep=set(sampled))
    assert len(ref["events"]) == 10240 and ref["summary"]["samples_total"] == 450560
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 2e-5
    acc = w0.astype(np.float64)
    for e in ref["events"]:
        acc -= sim.step_size(cfg, e["round"]) * gpu["U"][e["seq"]].astype(np.float64)
    assert np.abs(acc - gpu["w"]).max() <= 2e-6 * max(1.0, np.abs(acc).max())
    for k in range(0, 10240, 97):                     # update sums of the run itself (start models differ by fp32 round-off)
        assert rel_err(gpu["U"][k], ref["U"][k]) <= 1e-4, k
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for k in sampled:                             # restarted from the checker's start model
            e = ref["events"][k]
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][k])


def test_recycled_update_sums_give_the_same_model_bit_for_bit():
    # default handles reuse update-sum rows and snapshot slots during a run; a handle that keeps them all must agree
    cfg = workloads.get_config("cfg5", n_clients=300, n_rounds=6, data=dict(per_client=128))
    data, w0 = make(cfg)
    kept = run_gpu(cfg, data, w0, want_U=True)
    lean = run_gpu(cfg, data, w0, want_U=False)
    assert kept["w"].tobytes() == lean["w"].tobytes() and kept["blob"] == lean["blob"]
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run()
        with pytest.raises(api.AetError) as e:
            api.aet_get_update_sum(s.h, 0)
        assert e.value.status == 3                    # AET_ERR_STATE: rows were recycled


def test_cfg6_the_papers_setting_110_rounds_end_to_end():
    # Appendix Table 2 / A.2: 5 nodes, s_i = 10 i from round 1, eta_0 = 0.01, beta = 0.01, d = 1, uniform delays;
    # K = 60,000 iterations per node are 110 rounds (the count the paper prints), 61,050 samples per node
    cfg = workloads.get_config("cfg6")
    data, w0 = make(cfg)
    picks = {0, 137, 300, 549}
    ref = sim.run(cfg, data, w0, keep=picks)
    assert len(ref["events"]) == 550 and ref["summary"]["messages_up"] == 550
    assert ref["summary"]["messages_if_per_sample"] == 305250
    assert schedule.rounds_needed(60000, 10, 0, 1) == 110
    gpu = run_gpu(cfg, data, w0)
    f_gpu, f_ref = check_against_oracle(cfg, data, w0, gpu, ref)
    assert gpu["summary"]["messages_if_per_sample"] == 305250 and gpu["summary"]["messages_up"] == 550
    assert f_ref < np.log(10.0)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 2e-5
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for k in picks:
            e = ref["events"][k]
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][k])


@pytest.mark.parametrize("n_clients,l2", [(320, 0.0), (320, 1e-3), (480, 0.0), (480, 1e-3)])
def test_many_clients_take_the_kernel_variant_for_crowded_waves(n_clients, l2):
    # >= 296 round-tasks in a wave switch the kernel to its one-warp softmax
    cfg = workloads.get_config("cfg5", n_clients=n_clients, n_rounds=3, l2=l2, data=dict(per_client=64))
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0, keep=True)
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5
    for k in (0, 400, 3 * n_clients - 1):
        assert rel_err(gpu["U"][k], ref["U"][k]) <= 1e-4


@pytest.mark.parametrize("over", [
    dict(),                                                    # cfg5's step size: weak coupling, a few sweeps per block
    dict(flags=api.FLAG_STEPWISE_RECURRENCE),                  # the same walked step by step
    dict(lr=0.002),                                            # stronger coupling: more sweeps
    dict(lr=0.05, rounds_only=True),                           # coupling too strong for the sweeps: the kernel walks
    dict(sched_a=3, sched_b=1, n_rounds=9),                    # rounds of 1, 4, 7, ... samples: every tail length
    dict(max_lag_d=workloads.NEVER_WAIT, network_delay_mean=50.0, n_rounds=4),   # own sums in flight at round start
])
def test_tensor_memory_kernel_every_sampled_round_from_the_checkers_start_model(over):
    # more clients than SMs: the kernel that keeps U in tensor memory (tcgen05.mma, tf32 x 3); the single-round
    # parity call of such a handle runs that kernel too
    over = dict(dict(n_clients=200, n_rounds=6, data=dict(per_client=96)), **over)
    rounds_only = over.pop("rounds_only", False)
    cfg = workloads.get_config("cfg5", **over)
    data, w0 = make(cfg)
    if rounds_only:
        # 200 clients summed at this step size diverge end to end; the rounds themselves are well defined
        rng = np.random.default_rng(7)
        with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
            errs = [check_round_U(cfg, data, s.h, c, i, rng.normal(0, 0.05, size=w0.size))
                    for c, i in ((0, 0), (199, 5), (77, 3), (150, 1))]
        print("tensor-memory kernel per-round U errors: max %.1e" % max(errs))
        return
    ref = sim.run(cfg, data, w0, keep=True)
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 2e-5
    for k in range(0, len(ref["events"]), 23):
        assert rel_err(gpu["U"][k], ref["U"][k]) <= 1e-4, k
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        errs = [check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["seq"]])
                for e in ref["events"][::41]]
    print("tensor-memory kernel per-round U errors: max %.1e" % max(errs))


@pytest.mark.parametrize("over", [
    dict(max_lag_d=0), dict(max_lag_d=workloads.NEVER_WAIT, network_delay_mean=20.0),
    dict(n_clients=1), dict(lr_beta=0.05, l2=0.0), dict(delay_dist=1, n_stragglers=1, straggler_factor=30.0),
    dict(sched_a=3, sched_b=1, n_rounds=7),   # ragged: rounds of 1, 4, 7, ... samples
])
def test_variants_end_to_end(over):
    cfg = workloads.get_config("cfg1", data=dict(per_client=300), **over)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5


@pytest.mark.parametrize("over", [
    dict(sched_a=3, sched_b=1, n_rounds=9),                       # rounds of 1, 4, 7, ... 25 samples: every tail length
    dict(sched_a=1, sched_b=1, n_rounds=7, n_clients=3),          # rounds shorter than one block of 8
    dict(sched_a=5, sched_b=11, n_rounds=6, max_lag_d=0),         # odd sizes, everybody waits for everybody
    dict(n_clients=1, n_rounds=6),                                # one client: plain SGD
    dict(n_clients=2, n_rounds=6, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=500.0),   # own sums in flight
    dict(lr_beta=0.05, sched_a=7, sched_b=2),                     # step size changes from round to round
    dict(n_clients=330, n_rounds=4, sched_a=3, sched_b=2, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=50.0,
         data=dict(per_client=64)),   # more round-tasks than CTAs: a CTA runs several in a row, with sums in flight and ragged tails
])
def test_blocked_kernel_variants_without_l2(over):
    # lambda = 0 takes the kernel that runs eight steps per block; check ragged tails and start-model cases on it
    over = dict(over)
    cfg = workloads.get_config("cfg1", l2=0.0, data=over.pop("data", dict(per_client=300)), **over)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0, keep=True)
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5
    for k in range(0, len(ref["events"]), max(1, len(ref["events"]) // 40)):   # update sums of the run itself
        assert rel_err(gpu["U"][k], ref["U"][k]) <= 1e-4, k
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        worst = max(check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["seq"]])
                    for e in ref["events"][::max(1, len(ref["events"]) // 60)])
    assert worst <= U_TOL


@pytest.mark.parametrize("l2", [0.0, 1e-4])
def test_the_papers_schedule_shape_end_to_end(l2):
    # Table 2 / Appendix A.2 of the paper: five nodes, s_i = 10 i counted from round 1, eta_0 = 0.01 with
    # beta = 0.01 (step size constant within a round), d = 1; 12 rounds here instead of 110
    cfg = workloads.get_config("cfg1", n_clients=5, sched_a=10, sched_b=0, round_base=1, n_rounds=12, lr=0.01,
                               lr_beta=0.01, l2=l2, max_lag_d=1, data=dict(per_client=400))
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0, keep=True)
    assert [e["samples"] for e in ref["events"] if e["client"] == 0] == [10 * i for i in range(1, 13)]
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for e in ref["events"][::7]:
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["seq"]])


def test_many_own_updates_in_flight():
    # a slow network keeps several of a client's own sums in flight at round start
    cfg = workloads.get_config("cfg1", n_clients=2, n_rounds=6, max_lag_d=workloads.NEVER_WAIT,
                               network_delay_mean=500.0, data=dict(per_client=100))
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    assert max(e["round"] - sum(1 for f in ref["events"][:e["seen"]] if f["client"] == e["client"])
               for e in ref["events"]) >= 3
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5


def test_two_runs_are_bit_identical_and_reset_replays():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    a = run_gpu(cfg, data, w0)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run()
        w1 = s.model().copy()
        s.reset()
        s.run()
        w2 = s.model()
        blob, _ = s.log(raw=True)
    assert a["w"].tobytes() == w1.tobytes() == w2.tobytes()
    assert blob == a["blob"]
    assert all(u.tobytes() == v.tobytes() for u, v in zip(a["U"], run_gpu(cfg, data, w0)["U"]))


@pytest.mark.parametrize("n_clients", [6, 330])
def test_blocked_kernel_runs_are_bit_identical(n_clients):
    # 6 clients: the 8-warp instance (one round-task per SM); 330: the 4-warp instance, two CTAs per SM
    cfg = workloads.get_config("cfg1", l2=0.0, n_clients=n_clients, n_rounds=4, sched_a=5, sched_b=3,
                               data=dict(per_client=64))
    data, w0 = make(cfg)
    a = run_gpu(cfg, data, w0)
    b = run_gpu(cfg, data, w0)
    assert a["w"].tobytes() == b["w"].tobytes() and a["blob"] == b["blob"]
    assert all(u.tobytes() == v.tobytes() for u, v in zip(a["U"], b["U"]))


def test_run_in_two_calls_matches_the_checker_continued():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    r1 = sim.run(cfg, data, w0, n_rounds=2)
    r2 = sim.run(cfg, data, r1["w"], n_rounds=3, state=r1["state"])
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run(2)
        s.run(3)
        blob, summary = s.log(raw=True)
        w = s.model()
    assert blob == schedule.pack_events(r1["events"]) + schedule.pack_events(r2["events"])
    assert summary["samples_total"] == 600 and summary["t_end_ticks"] == r2["summary"]["t_end_ticks"]
    assert np.abs(w - r2["w"]).max() <= 1e-5


def test_host_buffers_are_accepted():
    cfg = workloads.get_config("cfg1", n_rounds=2)
    data, w0 = make(cfg)
    gpu_dev = run_gpu(cfg, data, w0)
    h = api.aet_create(cfg)
    try:
        api.aet_set_global_model(h, w0)
        for c, (x, y) in enumerate(data):
            api.aet_load_client_data(h, c, np.ascontiguousarray(x), np.ascontiguousarray(y))
        api.aet_run_rounds(h, 2)
        out = torch.empty(api.aet_n_params(h), dtype=torch.float32, device="cuda")
        api.aet_get_global_model(h, out)
        assert out.cpu().numpy().tobytes() == gpu_dev["w"].tobytes()
    finally:
        api.aet_destroy(h)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_handle_survives():
    cfg = workloads.get_config("cfg1", n_rounds=2)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        with pytest.raises(api.AetError) as e:
            api.aet_debug_wait_probe(s.h, 1 << 10)        # nothing ever signals that barrier
        assert e.value.status == 6                        # AET_ERR_TIMEOUT
        s.run()                                           # status was cleared; the context is intact
        assert np.abs(s.model() - ref["w"]).max() <= 1e-5
        with pytest.raises(api.AetError) as e:
            api.aet_debug_wait_probe(s.h, 0)
        assert e.value.status == 1


def test_zero_rounds_is_a_no_op():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run(0)
        events, summary = s.log()
        assert events == [] and summary["messages_up"] == 0
        assert s.model().tobytes() == w0.tobytes()


def test_errors_are_reported_not_raised_by_the_device():
    cfg = workloads.get_config("cfg1")
    data, w0 = make(cfg)
    h = api.aet_create(cfg)
    try:
        with pytest.raises(api.AetError) as e:
            api.aet_run_rounds(h, 1)                      # no client data yet
        assert e.value.status == 3
        x, y = to_device(data)[0]
        with pytest.raises(api.AetError) as e:
            api.aet_load_client_data(h, 9, x, y)          # client out of range
        assert e.value.status == 1
        with pytest.raises(api.AetError) as e:
            api.aet_set_global_model(h, w0[:100].copy())  # wrong length
        assert e.value.status == 1
        for c, (x, y) in enumerate(to_device(data)):
            api.aet_load_client_data(h, c, x, y)
        api.aet_run_rounds(h, 1)                          # and it still works afterwards
        assert len(api.aet_get_event_log(h)[0]) == 4
    finally:
        api.aet_destroy(h)
    with pytest.raises(api.AetError) as e:
        api.aet_create(workloads.get_config("cfg1", dims=[784, 64]))   # too many classes
    assert e.value.status == 2


@pytest.mark.parametrize("over", [
    dict(n_clients=5, sched_a=6, sched_b=2, l2=0.0),                                   # blocked kernel; some rounds are empty
    dict(n_clients=3, sched_a=10, sched_b=5, client_shares=[1, 2, 5], lr_beta=0.02, l2=1e-4),   # unequal p_c, step-by-step kernel
    dict(n_clients=200, sched_a=300, sched_b=200, l2=0.0, lr=1e-4, n_rounds=4, data=dict(per_client=64)),   # tensor-memory kernel
    dict(model=0, dims=[50, 10], n_clients=4, sched_a=5, sched_b=3, l2=0.0,
         data=dict(per_client=100, dim=50)),                                           # another width: the generic round kernel
])
def test_setup_split_of_a_global_round_size_end_to_end(over):
    # Algorithm 2: s_i = a i + b is the global size of round i, split among the nodes by coin flips
    base = dict(split_mode=1, n_rounds=7, data=dict(per_client=300))
    base.update(over)
    cfg = workloads.get_config("cfg1", **base)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0, keep=True)
    sizes = [e["samples"] for e in ref["events"]]
    assert len(set(sizes)) > 3 and ref["summary"]["samples_total"] == sum(
        cfg["sched_a"] * i + cfg["sched_b"] for i in range(cfg["n_rounds"]))
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert np.abs(gpu["w"] - ref["w"]).max() <= 1e-5
    for k, e in enumerate(ref["events"]):
        if e["samples"] == 0:
            assert not gpu["U"][k].any()                # an empty round sends a zero sum
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for e in ref["events"][::max(1, len(ref["events"]) // 25)]:
            if e["samples"]:
                check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["seq"]])
