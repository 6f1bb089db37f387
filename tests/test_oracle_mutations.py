"""Do the pins bite?  Each case plants one plausible mistake in the CPU checker
(never in the CUDA path) and expects the named pin to fail."""
import numpy as np
import pytest

import test_oracle_models as tm
import test_oracle_rng as tr
import test_oracle_schedule as ts
import test_oracle_sim as tsim
from oracle import models, rng, schedule, sim


def _fails(fn, *args):
    with pytest.raises((AssertionError, IndexError, ValueError, KeyError)):
        fn(*args)


def test_dropped_l2_term_is_caught(monkeypatch):
    real = models.loss_and_grad

    def no_l2_in_grad(w, X, y, dims, l2=0.0, precision=0):
        loss, _ = real(w, X, y, dims, l2, precision)
        return loss, real(w, X, y, dims, 0.0, precision)[1]
    monkeypatch.setattr(models, "loss_and_grad", no_l2_in_grad)
    _fails(tm.test_gradient_matches_central_differences, [9, 6, 10], 4, 0.05)
    _fails(tm.test_matches_torch_autograd_mlp)


def test_bias_gradient_scaled_wrongly_is_caught(monkeypatch):
    real = models.loss_and_grad

    def bad(w, X, y, dims, l2=0.0, precision=0):
        loss, g = real(w, X, y, dims, l2, precision)
        g = g.copy()
        g[-dims[-1]:] /= X.shape[0]
        return loss, g
    monkeypatch.setattr(models, "loss_and_grad", bad)
    _fails(tm.test_gradient_matches_central_differences, [7, 10], 5, 0.0)


def test_wrong_sign_of_the_local_step_is_caught(monkeypatch):
    real = sim.run_task

    def ascent(cfg, client_data, c, i, w_start):
        U, w_end = real(cfg, client_data, c, i, w_start)
        return U, 2 * np.asarray(w_start, dtype=np.float64) - w_end
    monkeypatch.setattr(sim, "run_task", ascent)
    _fails(tsim.test_update_sum_identity_U_equals_model_difference_over_eta)


def test_forgotten_in_flight_correction_is_caught(monkeypatch):
    real = sim.step_size
    calls = {"n": 0}

    # the correction is the only caller of step_size between a START and its run_task;
    # make own in-flight sums count for nothing by zeroing U rows through a patched run
    def run_without_correction(cfg, data, w0, n_rounds=None, keep=False, state=None):
        n_rounds = cfg["n_rounds"] if n_rounds is None else n_rounds
        events, summary, after = schedule.simulate(cfg, n_rounds, state)
        order = sorted([(e["t_apply"], 0, e["client"], e["round"], e) for e in events] +
                       [(e["t_start"], 1, e["client"], e["round"], e) for e in events], key=lambda r: r[:4])
        w_g = np.array(w0, dtype=np.float64)
        U = [None] * len(events)
        for _, kind, c, i, e in order:
            if kind == 1:
                U[e["seq"]] = sim.run_task(cfg, data[c], c, i, w_g.copy())[0]     # no own-update correction
            else:
                w_g -= real(cfg, i) * U[e["seq"]]
        return dict(events=events, summary=summary, w=w_g, U=U, w_start=[None] * len(events), state=after)
    monkeypatch.setattr(sim, "run", run_without_correction)
    _fails(tsim.test_one_client_is_plain_sgd_whatever_the_delays)


def test_start_before_apply_on_ties_is_caught(monkeypatch):
    monkeypatch.setattr(schedule, "APPLY", 1)
    monkeypatch.setattr(schedule, "START", 0)
    _fails(ts.test_apply_precedes_start_on_equal_ticks)


def test_round_size_off_by_one_is_caught(monkeypatch):
    monkeypatch.setattr(schedule, "sample_size", lambda a, b, i: a * (i + 1) + b)
    _fails(ts.test_round_counts_printed_in_the_paper, ("linear", 60000, 10, 0, 1, 110))
    _fails(ts.test_sample_totals_closed_form, "cfg2", 9300, 148800, 480)


def test_checkpoint_that_counts_the_client_itself_is_caught(monkeypatch):
    real = schedule.simulate

    def lenient(cfg, n_rounds, state=None):
        return real(dict(cfg, max_lag_d=schedule.NEVER_WAIT), n_rounds, state)
    monkeypatch.setattr(schedule, "simulate", lenient)
    _fails(ts.test_d0_every_client_waits_for_all_previous_rounds)
    _fails(ts.test_two_client_timeline_worked_by_hand)


def test_log2_instead_of_ln_is_caught(monkeypatch):
    monkeypatch.setattr(rng, "LN2_Q32", 1 << 32)
    _fails(tr.test_exp_scales_with_mean_and_floors_at_one_tick)
    _fails(tr.test_exp_draws_have_the_right_distribution)


def test_low_word_sample_index_is_caught(monkeypatch):
    monkeypatch.setattr(rng, "sample_index", lambda r, n: ((r & 0xFFFFFFFF) * n) >> 32)
    _fails(tsim.test_one_client_is_plain_sgd_whatever_the_delays)


def test_wrong_mixing_constant_is_caught(monkeypatch):
    real = rng.mix64
    monkeypatch.setattr(rng, "mix64", lambda z: real(z) ^ 1)
    _fails(tr.test_mix_matches_published_splitmix64_sequence)


def _with_source_edit(monkeypatch, old, new):
    """Plant a mistake in the checker's loss_and_grad by editing its source text."""
    import inspect
    src = inspect.getsource(models.loss_and_grad)
    assert src.count(old) == 1, old
    ns = dict(vars(models))
    exec(compile(src.replace(old, new), "<mutated loss_and_grad>", "exec"), ns)
    monkeypatch.setattr(models, "loss_and_grad", ns["loss_and_grad"])


@pytest.mark.parametrize("old,new", [
    ("A = [q(X)]", "A = [X]"),                                          # inputs not rounded
    ("Wq = [q(W) for W, _ in layers]", "Wq = [W for W, _ in layers]"),    # weights not rounded when read
    ("A.append(q(np.maximum(z, 0.0)))", "A.append(np.maximum(z, 0.0))"),  # activations not rounded
    ("gW[...] = A[l].T @ dZq", "gW[...] = A[l].T @ dZ"),                  # dZ unrounded in the weight gradient
    ("dA = dZq @ Wq[l].T", "dA = dZ @ Wq[l].T"),                          # dZ unrounded in the input gradient
    ("gb[...] = dZ.sum(axis=0)", "gb[...] = dZq.sum(axis=0)"),            # bias gradient from the rounded dZ
    ("z = A[l] @ Wq[l] + layers[l][1]", "z = q(A[l] @ Wq[l] + layers[l][1])"),   # logits / pre-activations rounded too
])
def test_a_moved_or_dropped_bf16_rounding_point_is_caught(monkeypatch, old, new):
    _with_source_edit(monkeypatch, old, new)
    _fails(tm.test_bf16_rounding_points_on_a_case_worked_by_hand)


def test_step_size_without_the_square_root_is_caught(monkeypatch):
    monkeypatch.setattr(schedule, "round_step_size", lambda lr, beta, t: lr / (1.0 + beta * t))
    _fails(ts.test_round_step_size_values_worked_by_hand)


def test_setup_split_that_reuses_the_coins_of_every_round_is_caught(monkeypatch):
    real = schedule.samples_before
    # coins keyed by the position inside the round only: every round replays the same coins
    monkeypatch.setattr(schedule, "split_round", lambda cfg, i: (
        lambda key, sh: [sum(1 for t in range(schedule.sample_size(cfg["sched_a"], cfg["sched_b"], i))
                             if schedule.assign_node(rng.draw(key, t), sh) == c) for c in range(cfg["n_clients"])])(
        rng.stream_key(cfg["seed"], rng.STREAM_SETUP, 0), schedule.client_shares(cfg)))
    _fails(ts.test_setup_split_uses_a_fresh_coin_for_every_iteration_of_every_round)


def test_setup_split_by_independent_draws_per_node_is_caught(monkeypatch):
    # each node flips its own coins: the expectation is right, the round total is not conserved
    def independent(cfg, i):
        n, sh = cfg["n_clients"], schedule.client_shares(cfg)
        s_i = schedule.sample_size(cfg["sched_a"], cfg["sched_b"], i)
        out = []
        for c in range(n):
            key = rng.stream_key(cfg["seed"], rng.STREAM_SETUP, c)
            out.append(sum(1 for t in range(s_i) if ((rng.draw(key, 1000 * i + t) >> 32) * sum(sh)) >> 32 < sh[c]))
        return out
    monkeypatch.setattr(schedule, "split_round", independent)
    _fails(ts.test_setup_split_conserves_every_round_and_reduces_to_one_node)


def test_ring_that_sends_to_every_node_is_caught(monkeypatch):
    import test_oracle_ring as tring
    monkeypatch.setattr(schedule, "ring_neighbours",
                        lambda n, c: [(k, v) for k, v in enumerate(w for w in range(n) if w != c)][:2] if n <= 3
                        else [(0, (c - 1) % n), (1, (c + 2) % n)])       # right-hand link skips a node
    _fails(tring.test_four_node_timeline_worked_by_hand)
    _fails(tring.test_node_model_is_w0_minus_own_and_neighbours_sums)


def test_ring_receive_with_the_receivers_step_size_is_caught(monkeypatch):
    import inspect
    import test_oracle_ring as tring
    src = inspect.getsource(sim.run_ring)
    old = 'W[c] -= step_size(cfg, q["round"], q["client"]) * U_by_task[q["task"]]'
    assert src.count(old) == 1
    ns = dict(vars(sim))
    exec(compile(src.replace(old, 'W[c] -= step_size(cfg, e["round"], c) * U_by_task[q["task"]]'), "<mutated run_ring>", "exec"), ns)
    monkeypatch.setattr(sim, "run_ring", ns["run_ring"])
    _fails(tring.test_node_model_is_w0_minus_own_and_neighbours_sums)


def test_ring_history_that_counts_at_round_start_instead_of_arrival_is_caught(monkeypatch):
    # Synchronize must see a message as soon as it arrives (the wait loop keeps tracking H); a history that only
    # moves when the node starts a round would leave the blocked node of the hand-worked timeline waiting for ever
    import inspect
    import test_oracle_ring as tring
    src = inspect.getsource(schedule.simulate_ring)
    old = "            H[node][sender] += 1\n"
    assert src.count(old) == 1
    ns = dict(vars(schedule))
    exec(compile(src.replace(old, "            H[node][sender] += 0\n"), "<mutated simulate_ring>", "exec"), ns)
    monkeypatch.setattr(schedule, "simulate_ring", ns["simulate_ring"])
    _fails(tring.test_four_node_timeline_worked_by_hand)


def test_cnn_pooling_gradient_without_the_quarter_is_caught(monkeypatch):
    monkeypatch.setattr(models, "_unpool", lambda g: np.repeat(np.repeat(g, 2, axis=2), 2, axis=3))
    _fails(tm.test_cnn_gradient_matches_central_differences, 0.0)
    _fails(tm.test_cnn_matches_torch_conv_pool_autograd)


def test_cnn_true_convolution_instead_of_correlation_is_caught(monkeypatch):
    real = models._windows
    monkeypatch.setattr(models, "_windows", lambda a: real(a)[..., ::-1, ::-1])
    _fails(tm.test_cnn_matches_torch_conv_pool_autograd)
    _fails(tm.test_cnn_one_bright_pixel_by_hand)
