"""GPU checks of the boundary's flags and status codes (every call through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import sim
from paper_2112_13935_b200 import api, workloads
from gpu_helpers import make, run_gpu, to_device

pytestmark = pytest.mark.gpu


def _small(**kw):
    return workloads.get_config("cfg1", n_rounds=3, data=dict(per_client=200), **kw)


@pytest.mark.parametrize("l2", [1e-4, 0.0])
def test_a_nan_pixel_is_reported_as_numeric_and_the_handle_stays_usable(l2):
    cfg = _small(l2=l2)
    data, w0 = make(cfg)
    ref = sim.run(cfg, data, w0)
    dev = to_device(data)
    bad = dev[2][0].clone()
    bad[:, 5] = float("nan")                             # whichever rows round 0 samples, one pixel is NaN
    out = np.full(w0.size, 7.0, dtype=np.float32)
    with api.Session(cfg, dev[:2] + [(bad, dev[2][1])] + dev[3:], torch.from_numpy(w0).cuda()) as s:
        s.run()
        with pytest.raises(api.AetError) as e:
            api.aet_get_global_model(s.h, out)
        assert e.value.status == 7 and (out == 7.0).all()    # AET_ERR_NUMERIC, out-parameter untouched
        api.aet_load_client_data(s.h, 2, *dev[2])            # the clean rows
        s.reset()
        s.run()
        assert np.abs(s.model() - ref["w"]).max() <= 1e-5


def test_borrowed_device_data_gives_the_run_of_copied_data_bit_for_bit():
    cfg = _small(l2=0.0, n_clients=6)
    data, w0 = make(cfg)
    copied = run_gpu(cfg, data, w0)
    borrowed = run_gpu(dict(cfg, flags=api.FLAG_BORROW_DATA), data, w0)
    assert copied["w"].tobytes() == borrowed["w"].tobytes() and copied["blob"] == borrowed["blob"]
    assert all(u.tobytes() == v.tobytes() for u, v in zip(copied["U"], borrowed["U"]))
    h = api.aet_create(dict(cfg, flags=api.FLAG_BORROW_DATA))
    try:
        with pytest.raises(api.AetError) as e:               # host memory cannot be borrowed
            api.aet_load_client_data(h, 0, np.ascontiguousarray(data[0][0]), np.ascontiguousarray(data[0][1]))
        assert e.value.status == 1
    finally:
        api.aet_destroy(h)
    with pytest.raises(api.AetError) as e:
        api.aet_create(dict(cfg, flags=1 << 9))              # unknown flag bit
    assert e.value.status == 2


@pytest.mark.parametrize("name,over", [("cfg1", dict(l2=1e-4)), ("cfg1", dict(l2=0.0)),
                                       ("cfg3", dict(n_clients=6, n_rounds=3, data=dict(total=1200)))])
def test_debug_checks_change_nothing_on_good_input_and_flag_a_bad_label(name, over):
    over = dict(over)
    cfg = workloads.get_config(name, **over) if name == "cfg3" else _small(**over)
    data, w0 = make(cfg)
    plain = run_gpu(cfg, data, w0, want_U=False)
    checked = run_gpu(dict(cfg, flags=api.FLAG_DEBUG_CHECKS), data, w0, want_U=False)
    assert plain["w"].tobytes() == checked["w"].tobytes() and plain["blob"] == checked["blob"]
    dev = to_device(data)
    y_bad = dev[1][1].clone()
    y_bad[3] = 10                                            # ten classes: 0..9
    h = api.aet_create(dict(cfg, flags=api.FLAG_DEBUG_CHECKS))
    try:
        api.aet_set_global_model(h, torch.from_numpy(w0).cuda())
        for c, (x, y) in enumerate(dev):
            api.aet_load_client_data(h, c, x, y_bad if c == 1 else y)
        with pytest.raises(api.AetError) as e:               # found while loading; reported at the next synchronising call
            api.aet_get_global_model(h)
        assert e.value.status == 3
        api.aet_load_client_data(h, 1, *dev[1])
        api.aet_run_rounds(h, cfg["n_rounds"])
        assert api.aet_get_global_model(h).tobytes() == plain["w"].tobytes()
    finally:
        api.aet_destroy(h)


@pytest.mark.parametrize("topology", [0, 1])
def test_prepared_schedule_gives_the_same_run(topology):
    # aet_prepare_rounds computes the schedule and the launch plan on a library thread under the data copies;
    # the run that follows uses them if the state still fits, and computes its own otherwise
    cfg = workloads.get_config("cfg1", topology=topology, n_clients=5, l2=0.0, data=dict(per_client=200))
    data, w0 = make(cfg)

    def run(prepare_for, rounds):
        h = api.aet_create(cfg)
        try:
            if prepare_for:
                api.aet_prepare_rounds(h, prepare_for)
            api.aet_set_global_model(h, w0)
            for c, (x, y) in enumerate(data):
                api.aet_load_client_data(h, c, x, y)
            for r in rounds:
                api.aet_run_rounds(h, r)
            blob, _ = api.aet_get_event_log(h, raw=True)
            W = [api.aet_get_node_model(h, c) for c in range(5)] if topology else [api.aet_get_global_model(h)]
        finally:
            api.aet_destroy(h)
        return blob, W

    plain = run(0, [3, 2])
    for prepared in (run(3, [3, 2]), run(4, [3, 2])):      # the plan that fits, and one for another run length
        assert prepared[0] == plain[0]
        assert all(a.tobytes() == b.tobytes() for a, b in zip(prepared[1], plain[1]))
    h = api.aet_create(cfg)                                # a thread still running when the handle goes away is waited for
    api.aet_prepare_rounds(h, 5)
    api.aet_destroy(h)
