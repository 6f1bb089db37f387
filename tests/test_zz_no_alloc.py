"""The entry point that allocates nothing, checked against the ordinary one.

Some callers may not allocate device memory while they run (their memory went
to a pool at start-up, or cudaMalloc's device-wide synchronisation is not
acceptable where they call from).  aet_round_no_alloc runs one round-task with
the kernel's scratch in an array built into the library.  This file is collected
last, so a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import sim
from paper_2112_13935_b200 import api, workloads
from gpu_helpers import U_TOL, make, rel_err, to_device

pytestmark = pytest.mark.gpu


def _cfg():
    return workloads.get_config("cfg3", n_clients=6, n_rounds=4, dims=[784, 48, 10], batch=16,
                                sched_a=16, sched_b=16, l2=1e-4, data=dict(total=1200))


def test_two_calls_in_a_row_match_the_ordinary_entry_point():
    cfg = _cfg()
    data, w0 = make(cfg)
    dev = to_device(data)
    P = w0.size
    rng = np.random.default_rng(3)
    with api.Session(cfg, dev, torch.from_numpy(w0).cuda()) as s:
        for client, rnd in ((2, 1), (5, 3)):           # two calls, back to back, different work
            w_in = (w0 + rng.normal(0, 0.01, size=P)).astype(np.float32)
            U_ref, w_ref = api.aet_debug_run_client_round(s.h, client, rnd, w_in)
            x, y = dev[client]
            w_dev = torch.from_numpy(w_in).cuda()
            U_dev = torch.full((P,), 7.0, dtype=torch.float32, device="cuda")   # stale contents must not leak
            wo_dev = torch.full((P,), 7.0, dtype=torch.float32, device="cuda")
            api.aet_round_no_alloc(cfg, client, rnd, x, y, w_dev, U_dev, wo_dev)
            torch.cuda.synchronize()
            assert rel_err(U_dev.cpu().numpy(), U_ref) <= U_TOL, (client, rnd)
            assert rel_err(wo_dev.cpu().numpy(), w_ref) <= U_TOL, (client, rnd)
            assert np.abs(U_ref).max() > 0


@pytest.mark.parametrize("name,over", [
    ("cfg1", dict(data=dict(per_client=300))),                                  # softmax regression, batch 1, l2 = 1e-4
    ("cfg3", dict(n_clients=6, n_rounds=4, data=dict(total=1200))),             # 784-128-10, batch 32
])
def test_shapes_the_handle_runs_on_specialised_kernels(name, over):
    # a handle gives these shapes to kernels of their own; the entry point that allocates nothing always runs the
    # generic one, so the two agree within rounding order - and both agree with the CPU checker
    cfg = workloads.get_config(name, **over)
    data, w0 = make(cfg)
    dev = to_device(data)
    P = w0.size
    rng = np.random.default_rng(5)
    with api.Session(cfg, dev, torch.from_numpy(w0).cuda()) as s:
        for client, rnd in ((1, 0), (3, 2), (0, 3)):
            w_in = (w0 + rng.normal(0, 0.01, size=P)).astype(np.float32)
            U_h, w_h = api.aet_debug_run_client_round(s.h, client, rnd, w_in)
            U_ref, w_ref = sim.run_task(cfg, data[client], client, rnd, w_in.astype(np.float64))
            x, y = dev[client]
            U_dev = torch.full((P,), 7.0, dtype=torch.float32, device="cuda")
            wo_dev = torch.full((P,), 7.0, dtype=torch.float32, device="cuda")
            api.aet_round_no_alloc(cfg, client, rnd, x, y, torch.from_numpy(w_in).cuda(), U_dev, wo_dev)
            torch.cuda.synchronize()
            for got_U, got_w in ((U_dev.cpu().numpy(), wo_dev.cpu().numpy()), (U_h, w_h)):
                assert rel_err(got_U, U_ref) <= U_TOL, (client, rnd)
                assert rel_err(got_w, w_ref) <= U_TOL, (client, rnd)


def test_requests_beyond_the_fixed_scratch_are_refused():
    big = workloads.get_config("cfg4", precision=0)    # 820,874 parameters
    dummy = torch.zeros(64, dtype=torch.float32, device="cuda")
    lab = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(api.AetError) as e:
        api.aet_round_no_alloc(big, 0, 0, dummy.view(1, 64).expand(64, 64).contiguous(), lab, dummy, dummy, dummy)
    assert e.value.status == 2 and "too large" in str(e.value)
    with pytest.raises(api.AetError) as e:
        api.aet_round_no_alloc(workloads.get_config("cfg4", dims=[64, 16, 10]), 0, 0,
                               dummy.view(1, 64).expand(64, 64).contiguous(), lab, dummy, dummy, dummy)
    assert e.value.status == 2                          # precision 1 is not offered here
