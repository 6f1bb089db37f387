"""The multi-GPU plumbing (replicas only) exercised with two gloo ranks on CPU."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2112_13935_b200 import api, dist, workloads
    r, w, _ = dist.init_from_env("gloo")
    # each rank is an independent replica with its own seed: schedules differ
    cfg = workloads.get_config("cfg1", seed=r)
    events, summary = api.aet_schedule_only(cfg, 5)
    dist.barrier()
    rate = dist.job_throughput(summary["samples_total"], 1.0 + r)
    out.put((r, w, summary["samples_total"], events[0]["t_trigger"], rate,
             dist.max_over_ranks(float(r)), dist.sum_over_ranks(1.0)))
    dist.shutdown()


def test_two_replicas_aggregate_counts_and_take_the_slowest_time():
    from paper_2112_13935_b200 import build
    build.build()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, w0, s0, t0, rate0, mx0, sm0), (r1, w1, s1, t1, rate1, mx1, sm1) = res
    assert (r0, r1, w0, w1) == (0, 1, 2, 2)
    assert s0 == s1 == 600 and t0 != t1          # same work, different seeds
    assert rate0 == rate1 == 1200 / 2.0          # all units / slowest rank's time
    assert mx0 == mx1 == 1.0 and sm0 == sm1 == 2.0
