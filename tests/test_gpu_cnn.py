"""GPU parity of the small convolutional classifier (LeNet shape) against the CPU checker."""
import numpy as np
import pytest
import torch

from oracle import sim
from paper_2112_13935_b200 import api, workloads
from gpu_helpers import check_against_oracle, check_round_U, make, rel_err, run_gpu, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("over", [
    dict(dims=[16, 1, 4, 6, 12, 10, 10], batch=4, sched_a=4, sched_b=4, data=dict(total=600, dim=256)),            # small maps
    dict(dims=[16, 2, 3, 5, 9, 8, 10], batch=3, sched_a=3, sched_b=6, l2=1e-3, data=dict(total=600, dim=512)),     # two input planes, l2
    dict(n_rounds=3, data=dict(total=800)),                                                                        # the LeNet shape itself
    dict(n_rounds=4, n_clients=3, max_lag_d=workloads.NEVER_WAIT, network_delay_mean=300.0, batch=8, sched_a=8, sched_b=8,
         data=dict(total=600)),                                                                                    # own sums in flight
    dict(topology=1, n_rounds=3, n_clients=4, data=dict(total=600)),                                               # on the ring
    dict(n_rounds=2, n_clients=40, data=dict(total=2400)),   # fuller launch: clusters of 2, rows in shared memory, activations in scratch
    dict(n_rounds=2, n_clients=80, data=dict(total=4000)),   # one CTA per round-task, nothing staged beside the model
])
def test_conv_classifier_end_to_end_and_round_U(over):
    base = dict(n_clients=4, n_rounds=4)
    base.update(over)
    cfg = workloads.get_config("cfg7", **base)
    data, w0 = make(cfg)
    assert w0.size == workloads.model_n_params(cfg)
    if cfg.get("topology"):
        from test_gpu_ring import check_ring, run_ring_gpu
        ref = sim.run_ring(cfg, data, w0, keep=True)
        gpu = run_ring_gpu(cfg, data, w0)
        assert gpu["blob"] == __import__("oracle").schedule.pack_ring_events(ref["deliveries"])
        for c in range(cfg["n_clients"]):
            assert rel_err(gpu["W"][c], ref["W"][c]) <= 2e-5
        starts = [(e["client"], e["round"], ref["w_start"][e["task"]]) for e in ref["tasks"][::3]]
    else:
        ref = sim.run(cfg, data, w0, keep=True)
        gpu = run_gpu(cfg, data, w0)
        check_against_oracle(cfg, data, w0, gpu, ref)
        assert rel_err(gpu["w"], ref["w"]) <= 2e-5
        starts = [(e["client"], e["round"], ref["w_start"][e["seq"]]) for e in ref["events"][::3]]
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        errs = [check_round_U(cfg, data, s.h, c, i, w) for c, i, w in starts]
    print("conv classifier per-round U errors: max %.1e" % max(errs))


def test_conv_runs_are_bit_identical():
    # clusters of 8 sum their partial gradients in rank order and push the new weights into every copy between
    # two cluster barriers: nothing may depend on timing
    cfg = workloads.get_config("cfg7", n_clients=6, n_rounds=3, data=dict(total=1200))
    data, w0 = make(cfg)
    a = run_gpu(cfg, data, w0)
    b = run_gpu(cfg, data, w0)
    assert a["w"].tobytes() == b["w"].tobytes() and a["blob"] == b["blob"]
    assert all(u.tobytes() == v.tobytes() for u, v in zip(a["U"], b["U"]))


def test_cfg7_full_size_against_the_checker():
    # 16 clients, LeNet shape on 60,000 28x28 images, minibatch 16, s_i = 32 i + 32 for 12 rounds: 39,936 samples
    cfg = workloads.get_config("cfg7")
    data, w0 = make(cfg)
    picks = {0, 90, 191}
    ref = sim.run(cfg, data, w0, keep=picks)
    assert len(ref["events"]) == 192 and ref["summary"]["samples_total"] == 39936
    gpu = run_gpu(cfg, data, w0)
    check_against_oracle(cfg, data, w0, gpu, ref)
    assert rel_err(gpu["w"], ref["w"]) <= 1e-4
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        for k in picks:
            e = ref["events"][k]
            check_round_U(cfg, data, s.h, e["client"], e["round"], ref["w_start"][k])


def test_conv_shapes_the_kernel_cannot_run_are_refused():
    for dims in ([15, 1, 4, 6, 12, 10, 10], [28, 1, 6, 16, 400, 84, 10], [12, 1, 4, 6, 12, 10, 10]):
        with pytest.raises(api.AetError) as e:
            api.aet_create(workloads.get_config("cfg7", dims=dims))
        assert e.value.status == 2, dims
