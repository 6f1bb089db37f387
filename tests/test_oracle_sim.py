"""Pins for the whole-run checker: special cases the paper states in prose, the
server rule, the two-client timeline worked by hand and a convex problem."""
import numpy as np
import pytest
from scipy import optimize

from oracle import models, rng, schedule, sim
from paper_2112_13935_b200 import workloads
from test_oracle_schedule import hand_cfg


def _small(name="cfg1", per_client=60, **kw):
    cfg = workloads.get_config(name, data=dict(per_client=per_client), **kw)
    return cfg, workloads.make_client_data(cfg), workloads.make_start_model(cfg)


def test_update_sum_identity_U_equals_model_difference_over_eta():
    # Algorithm 3: w -= eta g and U += g in the same loop, so U = (w_start - w_end) / eta.
    cfg, data, w0 = _small()
    U, w_end = sim.run_task(cfg, data[1], 1, 2, w0)
    np.testing.assert_allclose(U, (w0 - w_end) / sim.step_size(cfg, 2), rtol=1e-9, atol=1e-12)
    assert np.abs(U).max() > 0


def test_one_client_is_plain_sgd_whatever_the_delays():
    # Appendix: with n = 1 the framework "works as the traditional SGD method".
    for net in (0.5, 50.0):
        cfg, data, w0 = _small(n_clients=1, network_delay_mean=net, n_rounds=4)
        out = sim.run(cfg, data, w0)
        X, y = data[0]
        key = rng.stream_key(cfg["seed"], rng.STREAM_SAMPLE, 0)
        w = w0.astype(np.float64)
        eta, lam = float(np.float32(cfg["lr"])), float(np.float32(cfg["l2"]))
        for k in range(out["summary"]["samples_total"]):
            j = ((rng.draw(key, k) >> 32) * len(y)) >> 32
            x = X[j].astype(np.float64)
            z = x @ w[:7840].reshape(784, 10) + w[7840:]
            p = np.exp(z - z.max())
            p /= p.sum()
            p[y[j]] -= 1.0
            g = np.concatenate([(np.outer(x, p) + lam * w[:7840].reshape(784, 10)).ravel(), p])
            w = w - eta * g
        np.testing.assert_allclose(out["w"], w, rtol=1e-11, atol=1e-13)


def test_global_model_is_w0_minus_applied_updates():
    # Definition 1 / Receive: w = w_0 - sum eta_k U_k over the applied updates.
    cfg, data, w0 = _small(lr_beta=0.01)
    out = sim.run(cfg, data, w0)
    acc = w0.astype(np.float64)
    for e in out["events"]:
        acc = acc - sim.step_size(cfg, e["round"]) * out["U"][e["seq"]]
    np.testing.assert_allclose(out["w"], acc, rtol=1e-12, atol=1e-14)
    etas = {sim.step_size(cfg, i) for i in range(5)}
    assert len(etas) == 5 and max(etas) == float(np.float32(0.01))


def test_d0_is_synchronous_local_sgd_independent_of_delay_seed():
    # Appendix: d = 0 makes all nodes wait for each other, so every round starts
    # from the common model and the result does not depend on the delays.
    results = []
    for seed_shift, net in ((0, 0.5), (0, 5.0)):
        cfg, data, w0 = _small(max_lag_d=0, n_rounds=3, network_delay_mean=net)
        results.append(sim.run(cfg, data, w0)["w"])
    cfg, data, w0 = _small(max_lag_d=0, n_rounds=3)
    w = w0.astype(np.float64)
    for i in range(3):
        total = sum(sim.run_task(cfg, data[c], c, i, w)[0] for c in range(4))
        w = w - sim.step_size(cfg, i) * total
    np.testing.assert_allclose(results[0], w, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(results[1], w, rtol=1e-11, atol=1e-13)


def test_start_models_of_the_hand_worked_timeline():
    cfg = hand_cfg()
    cfg["data"]["per_client"] = 30
    data, w0 = workloads.make_client_data(cfg), workloads.make_start_model(cfg)
    out = sim.run(cfg, data, w0, keep=True)
    U, eta = out["U"], float(np.float32(cfg["lr"]))
    seq = {(e["client"], e["round"]): e["seq"] for e in out["events"]}
    assert seq == {(0, 0): 0, (0, 1): 1, (1, 0): 2, (0, 2): 3, (1, 1): 4, (1, 2): 5}
    w0 = w0.astype(np.float64)
    want = {
        (0, 0): w0, (1, 0): w0,
        (0, 1): w0 - eta * U[0],                              # own round 0 still in flight
        (1, 1): w0 - eta * U[0] - eta * U[2],                 # seen {0}; own (1,0) in flight
        (0, 2): w0 - eta * (U[0] + U[1] + U[2]),              # seen {0,1,2}
        (1, 2): w0 - eta * (U[0] + U[1] + U[2] + U[3] + U[4]),  # seen {0..3}; own (1,1) in flight
    }
    for key, w in want.items():
        np.testing.assert_allclose(out["w_start"][seq[key]], w, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(out["w"], w0 - eta * sum(U), rtol=1e-12, atol=1e-14)


def test_local_models_follow_receive_and_end_equal_to_the_global_model():
    # Paper form: each node keeps w_c, adds received sums (Receive) and its own
    # steps; Section 5: all nodes end at the same solution.
    cfg, data, w0 = _small(n_rounds=4, n_stragglers=1, straggler_factor=5.0)
    out = sim.run(cfg, data, w0, keep=True)
    ev = out["events"]
    for c in range(cfg["n_clients"]):
        mine = sorted((e for e in ev if e["client"] == c), key=lambda e: e["round"])
        w_c, seen_before = w0.astype(np.float64), 0
        for e in mine:
            for f in ev[seen_before:e["seen"]]:
                if f["client"] != c:
                    w_c = w_c - sim.step_size(cfg, f["round"]) * out["U"][f["seq"]]
            seen_before = e["seen"]
            np.testing.assert_allclose(w_c, out["w_start"][e["seq"]], rtol=1e-10, atol=1e-13)
            w_c = w_c - sim.step_size(cfg, e["round"]) * out["U"][e["seq"]]
        for f in ev[seen_before:]:
            if f["client"] != c:
                w_c = w_c - sim.step_size(cfg, f["round"]) * out["U"][f["seq"]]
        np.testing.assert_allclose(w_c, out["w"], rtol=1e-10, atol=1e-13)


def test_convex_case_approaches_the_brute_force_optimum():
    cfg = workloads.get_config("cfg1", n_clients=1, l2=0.05, lr=0.05, lr_beta=0.05, n_rounds=30,
                               data=dict(per_client=200))
    data, w0 = workloads.make_client_data(cfg), workloads.make_start_model(cfg)
    dims, lam = cfg["dims"], float(np.float32(cfg["l2"]))
    X, y = data[0]

    def fg(w):
        return models.loss_and_grad(w, X, y, dims, lam)
    best = optimize.minimize(fg, w0.astype(np.float64), jac=True, method="L-BFGS-B",
                             options=dict(maxiter=5000, ftol=1e-15, gtol=1e-10))
    f_star = best.fun
    assert np.abs(fg(best.x)[1]).max() < 1e-6
    gaps = []
    for R in (5, 15, 30):
        w = sim.run(cfg, data, w0, n_rounds=R)["w"]
        gaps.append(models.full_loss(w, data, dims, lam) - f_star)
    assert all(g > 0 for g in gaps)
    assert gaps[0] > gaps[1] > gaps[2]
    assert gaps[2] < 0.05 * (models.full_loss(w0, data, dims, lam) - f_star)


def test_minibatch_mlp_run_is_consistent():
    cfg = workloads.get_config("cfg3", n_clients=3, n_rounds=2, batch=4, sched_a=4, sched_b=4,
                               dims=[784, 16, 10], data=dict(total=300))
    data, w0 = workloads.make_client_data(cfg), workloads.make_start_model(cfg)
    out = sim.run(cfg, data, w0)
    assert [e["steps"] for e in out["events"] if e["round"] == 1] == [2, 2, 2]
    acc = w0.astype(np.float64) - float(np.float32(cfg["lr"])) * sum(out["U"])
    np.testing.assert_allclose(out["w"], acc, rtol=1e-12, atol=1e-14)
    assert models.full_loss(out["w"], data, cfg["dims"]) < models.full_loss(w0, data, cfg["dims"])
