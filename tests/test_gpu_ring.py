"""GPU parity of the peer-to-peer ring (every node its own model, sums to the two neighbours only)
against the CPU checker.  Every call goes through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import models, schedule, sim
from paper_2112_13935_b200 import api, workloads
from gpu_helpers import LOSS_TOL, U_TOL, check_round_U, make, rel_err, to_device

pytestmark = pytest.mark.gpu


def run_ring_gpu(cfg, data, w0, n_rounds=None, calls=None):
    if not calls:   # the update sums are read back below: their rows must not be recycled
        cfg = dict(cfg, flags=cfg.get("flags", 0) | api.FLAG_KEEP_UPDATE_SUMS)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for r in (calls or [n_rounds]):
            s.run(r)
        blob, summary = s.log(raw=True)
        n_tasks = cfg["n_clients"] * sum(calls) if calls else cfg["n_clients"] * (n_rounds or cfg["n_rounds"])
        W = [api.aet_get_node_model(s.h, c) for c in range(cfg["n_clients"])]
        U = None if calls else [api.aet_get_update_sum(s.h, k) for k in range(n_tasks)]
        with pytest.raises(api.AetError) as e:
            api.aet_get_global_model(s.h)
        assert e.value.status == 3                     # no server model in this topology
    return dict(blob=blob, summary=summary, W=W, U=U)


def check_ring(cfg, data, gpu, ref, w_tol=1e-5):
    assert gpu["blob"] == schedule.pack_ring_events(ref["deliveries"]), "delivery log differs"
    assert gpu["summary"] == ref["summary"]
    dims, l2, prec = cfg["dims"], sim.f32(cfg["l2"]), cfg["precision"]
    for c in range(cfg["n_clients"]):
        assert np.abs(gpu["W"][c] - ref["W"][c]).max() <= w_tol * max(1.0, np.abs(ref["W"][c]).max()), c
        f_gpu = models.full_loss(gpu["W"][c], data, dims, l2, prec)
        f_ref = models.full_loss(ref["W"][c], data, dims, l2, prec)
        assert abs(f_gpu - f_ref) <= LOSS_TOL, (c, f_gpu, f_ref)


@pytest.mark.parametrize("over", [
    dict(n_clients=5, l2=1e-4), dict(n_clients=5, l2=0.0), dict(n_clients=1, l2=0.0), dict(n_clients=2, l2=0.0),
    dict(n_clients=6, l2=0.0, max_lag_d=0, n_stragglers=1, straggler_factor=10.0),
    dict(n_clients=7, l2=0.0, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=40.0, lr_beta=0.05),
    dict(n_clients=4, l2=0.0, split_mode=1, sched_a=9, sched_b=4, client_shares=[3, 1, 1, 2]),
    dict(n_clients=200, l2=0.0, lr=1e-4, sched_a=8, sched_b=8, n_rounds=4, data=dict(per_client=64)),   # crowded: tensor-memory kernel
])
def test_ring_softmax_regression_end_to_end(over):
    base = dict(topology=1, n_rounds=6, data=dict(per_client=200))
    base.update(over)
    cfg = workloads.get_config("cfg1", **base)
    data, w0 = make(cfg)
    ref = sim.run_ring(cfg, data, w0, keep=True)
    gpu = run_ring_gpu(cfg, data, w0)
    check_ring(cfg, data, gpu, ref)
    for e in ref["tasks"][::max(1, len(ref["tasks"]) // 30)]:
        if e["samples"]:
            assert rel_err(gpu["U"][e["task"]], ref["U"][e["task"]]) <= 1e-4, e["task"]
    # the invariant at any size: a node's model is w_0 minus its own and its neighbours' applied sums
    n = cfg["n_clients"]
    for c in range(min(n, 6)):
        acc = w0.astype(np.float64)
        for e in ref["tasks"]:
            if e["client"] in {(c - 1) % n, c, (c + 1) % n}:
                acc -= sim.step_size(cfg, e["round"], e["client"]) * gpu["U"][e["task"]].astype(np.float64)
        assert np.abs(acc - gpu["W"][c]).max() <= 3e-6 * max(1.0, np.abs(acc).max())
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for e in ref["tasks"][::max(1, len(ref["tasks"]) // 12)]:
            if e["samples"]:
                check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["task"]])


def test_ring_mlp_end_to_end():
    cfg = workloads.get_config("cfg3", topology=1, n_clients=6, n_rounds=4, data=dict(total=1200))
    data, w0 = make(cfg)
    ref = sim.run_ring(cfg, data, w0, keep=True)
    gpu = run_ring_gpu(cfg, data, w0)
    check_ring(cfg, data, gpu, ref, w_tol=2e-5)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for e in ref["tasks"][::5]:
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][e["task"]])


def test_ring_run_in_two_calls_matches_the_checker_continued():
    cfg = workloads.get_config("cfg1", topology=1, n_clients=5, l2=0.0, data=dict(per_client=200))
    data, w0 = make(cfg)
    r1 = sim.run_ring(cfg, data, w0, n_rounds=2)
    r2 = sim.run_ring(cfg, data, w0, n_rounds=3, state=r1["state"], node_models=r1["W"])
    gpu = run_ring_gpu(cfg, data, w0, calls=[2, 3])
    assert gpu["blob"] == schedule.pack_ring_events(r1["deliveries"]) + schedule.pack_ring_events(r2["deliveries"])
    for c in range(5):
        assert np.abs(gpu["W"][c] - r2["W"][c]).max() <= 1e-5


def test_the_papers_ring_experiment_setting_110_rounds():
    # Appendix Table 2: 5 compute nodes on a ring, s_i = 10 i from round 1, eta_0 = 0.01, beta = 0.01, d = 1,
    # uniform delays; 110 communication rounds for K = 60,000 iterations per node
    cfg = workloads.get_config("cfg6", topology=1)
    data, w0 = make(cfg)
    ref = sim.run_ring(cfg, data, w0, keep={0, 250, 549})
    assert len(ref["tasks"]) == 550 and ref["summary"]["messages_up"] == 1100
    gpu = run_ring_gpu(cfg, data, w0)
    check_ring(cfg, data, gpu, ref, w_tol=2e-5)
    # the node models differ (sums are not forwarded) but every one of them matched the checker's above
    losses = [models.full_loss(w, data, cfg["dims"]) for w in gpu["W"]]
    assert np.isfinite(losses).all()
    print("ring node losses:", ["%.3f" % v for v in losses])
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for k in (0, 250, 549):
            e = ref["tasks"][k]
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][k])


@pytest.mark.parametrize("name, over", [
    ("cfg6", dict(n_rounds=30)),
    ("cfg3", dict(n_clients=6, n_rounds=4, data=dict(total=1800))),
])
def test_ring_with_recycled_rows_equals_ring_with_kept_rows(name, over):
    # without AET_FLAG_KEEP_UPDATE_SUMS a row of the update-sum array is written again once its last Receive has run
    cfg = workloads.get_config(name, topology=1, **over)
    data, w0 = make(cfg)
    kept = run_ring_gpu(cfg, data, w0)                                   # sets the flag: one row per round-task
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run(cfg["n_rounds"])
        blob, _ = s.log(raw=True)
        W = [api.aet_get_node_model(s.h, c) for c in range(cfg["n_clients"])]
        with pytest.raises(api.AetError) as e:
            api.aet_get_update_sum(s.h, 0)
        assert e.value.status == 3
    assert blob == kept["blob"]
    for c in range(cfg["n_clients"]):
        assert W[c].tobytes() == kept["W"][c].tobytes()
