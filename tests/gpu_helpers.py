"""Shared pieces of the GPU parity tests (every call goes through the C ABI)."""
import numpy as np
import torch

from oracle import models, schedule, sim
from paper_2112_13935_b200 import api, workloads

U_TOL = 1e-5      # max_j |U_gpu - U_ref| / max_j |U_ref| per round-task (fp32 paths)
LOSS_TOL = 1e-3   # |F(w_gpu) - F(w_ref)|, F evaluated by the checker in fp64


def to_device(data):
    return [(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()) for x, y in data]


def make(cfg):
    data = workloads.make_client_data(cfg)
    w0 = workloads.make_start_model(cfg)
    return data, w0


def rel_err(got, want):
    want = np.asarray(want, dtype=np.float64)
    return float(np.abs(np.asarray(got, dtype=np.float64) - want).max() / max(np.abs(want).max(), 1e-300))


def run_gpu(cfg, data, w0, n_rounds=None, want_U=True):
    if want_U:   # update sums are recycled during a run unless the handle is told to keep them
        cfg = dict(cfg, flags=cfg.get("flags", 0) | api.FLAG_KEEP_UPDATE_SUMS)
    with api.Session(cfg, to_device(data), torch.from_numpy(w0).cuda()) as s:
        s.run(n_rounds)
        blob, summary = s.log(raw=True)
        w = s.model()
        n = len(blob) // 64
        U = [api.aet_get_update_sum(s.h, k) for k in range(n)] if want_U else None
        stats = api.aet_get_stats(s.h)
    return dict(blob=blob, summary=summary, w=w, U=U, stats=stats)


def check_against_oracle(cfg, data, w0, gpu, ref, u_tol=U_TOL, loss_tol=LOSS_TOL):
    assert gpu["blob"] == schedule.pack_events(ref["events"]), "event log differs"
    assert gpu["summary"] == ref["summary"]
    dims, l2, prec = cfg["dims"], sim.f32(cfg["l2"]), cfg["precision"]
    if cfg["model"] == 2:
        f_gpu = models.cnn_full_loss(gpu["w"], data, dims, l2)
        f_ref = models.cnn_full_loss(ref["w"], data, dims, l2)
    else:
        f_gpu = models.full_loss(gpu["w"], data, dims, l2, prec)
        f_ref = models.full_loss(ref["w"], data, dims, l2, prec)
    assert abs(f_gpu - f_ref) <= loss_tol, (f_gpu, f_ref)
    return f_gpu, f_ref


def check_round_U(cfg, data, h, c, i, w_start, u_tol=U_TOL, flip_frac=0.0, flip_tol=None):
    """Round-task (c, i) restarted on both sides from the same fp32 model.

    Entry by entry |U_gpu - U_or| / max|U_or| must stay within ``u_tol``.  Where the arithmetic takes discrete
    decisions whose inputs differ by accumulation order (a bf16 rounding, a ReLU mask), ``flip_tol`` admits a
    share ``flip_frac`` of the entries above ``u_tol``, none of them above ``flip_tol``."""
    w32 = np.ascontiguousarray(w_start, dtype=np.float32)
    U_gpu, w_gpu = api.aet_debug_run_client_round(h, c, i, w32)
    U_ref, w_ref = sim.run_task(cfg, data[c], c, i, w32.astype(np.float64))
    d = np.abs(U_gpu - U_ref) / np.abs(U_ref).max()
    eu, ew = float(d.max()), rel_err(w_gpu, w_ref)
    if flip_tol is None:
        assert eu <= u_tol, (c, i, eu)
    else:
        share = float((d > u_tol).mean())
        assert share <= flip_frac, (c, i, share, eu)
        assert eu <= flip_tol, (c, i, eu)
    assert ew <= u_tol, (c, i, ew)
    return eu
