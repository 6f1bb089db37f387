"""Thin Python binding of the C ABI in include/aet.h (same names, marshalling only).

torch supplies device memory, pinned host memory and the stream; every step of
the method runs inside the library's kernels and host scheduler.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import _lib
from ._lib import AetConfig, AetEvent, AetStats, AetSummary, NEVER_WAIT, STATUS_NAMES  # noqa: F401

FLAG_BORROW_DATA, FLAG_DEBUG_CHECKS, FLAG_KEEP_UPDATE_SUMS, FLAG_STEPWISE_RECURRENCE = 1, 2, 4, 8   # AET_FLAG_*


class AetError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {message}")
        self.status = status


def make_config(cfg: dict) -> AetConfig:
    """A workload dict (see workloads.CONFIGS) as the library's aet_config."""
    c = AetConfig()
    c.struct_size = C.sizeof(AetConfig)
    dims = list(cfg["dims"])
    c.n_layers = len(dims) - 1
    for i, d in enumerate(dims):
        c.dims[i] = d
    for name, _ in AetConfig._fields_:
        if name in ("struct_size", "n_layers", "dims", "flags", "split_mode", "topology", "client_shares"):
            continue
        setattr(c, name, cfg[name])
    c.flags = int(cfg.get("flags", 0))
    c.split_mode = int(cfg.get("split_mode", 0))
    c.topology = int(cfg.get("topology", 0))
    shares = cfg.get("client_shares")
    if shares:
        arr = (C.c_uint32 * len(shares))(*[int(v) for v in shares])
        c.client_shares = C.cast(arr, C.POINTER(C.c_uint32))
        c._shares_keepalive = arr      # the library copies them in aet_create; until then they live here
    return c


def _ptr(buf):
    """Address of a torch tensor, numpy array or raw int; None -> null."""
    if buf is None:
        return None
    if isinstance(buf, int):
        return C.c_void_p(buf)
    if isinstance(buf, np.ndarray):
        assert buf.flags["C_CONTIGUOUS"]
        return C.c_void_p(buf.ctypes.data)
    assert buf.is_contiguous()
    return C.c_void_p(buf.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return C.c_void_p(stream if isinstance(stream, int) else stream.cuda_stream)


def _check(handle, status):
    if status != 0:
        msg = _lib.load().aet_last_error(handle)
        raise AetError(status, msg.decode() if msg else "")


def aet_create(cfg) -> C.c_void_p:
    conf = cfg if isinstance(cfg, AetConfig) else make_config(cfg)
    h = C.c_void_p()
    _check(None, _lib.load().aet_create(C.byref(conf), C.byref(h)))
    return h


def aet_destroy(h):
    _check(h, _lib.load().aet_destroy(h))


def aet_reset(h, stream=None):
    _check(h, _lib.load().aet_reset(h, _stream(stream)))


def aet_set_global_model(h, w0, stream=None):
    _check(h, _lib.load().aet_set_global_model(h, _ptr(w0), w0.size if isinstance(w0, np.ndarray) else w0.numel(),
                                               _stream(stream)))


def aet_load_client_data(h, client: int, x, y, stream=None):
    n = x.shape[0]
    _check(h, _lib.load().aet_load_client_data(h, client, _ptr(x), _ptr(y), n, _stream(stream)))


def aet_run_rounds(h, n_rounds: int, stream=None):
    _check(h, _lib.load().aet_run_rounds(h, n_rounds, _stream(stream)))


def aet_prepare_rounds(h, n_rounds: int):
    """Start the host-side schedule and launch plan of the next aet_run_rounds(h, n_rounds) on a library thread."""
    _check(h, _lib.load().aet_prepare_rounds(h, n_rounds))


def aet_n_params(h) -> int:
    return int(_lib.load().aet_n_params(h))


def aet_get_global_model(h, out=None, stream=None):
    if out is None:
        out = np.empty(aet_n_params(h), dtype=np.float32)
    n = out.size if isinstance(out, np.ndarray) else out.numel()
    _check(h, _lib.load().aet_get_global_model(h, _ptr(out), n, _stream(stream)))
    return out


def aet_get_node_model(h, node: int, out=None, stream=None):
    if out is None:
        out = np.empty(aet_n_params(h), dtype=np.float32)
    n = out.size if isinstance(out, np.ndarray) else out.numel()
    _check(h, _lib.load().aet_get_node_model(h, node, _ptr(out), n, _stream(stream)))
    return out


def aet_get_update_sum(h, seq: int, out=None, stream=None):
    if out is None:
        out = np.empty(aet_n_params(h), dtype=np.float32)
    n = out.size if isinstance(out, np.ndarray) else out.numel()
    _check(h, _lib.load().aet_get_update_sum(h, seq, _ptr(out), n, _stream(stream)))
    return out


def _events_from(arr, n):
    names = [f for f, _ in AetEvent._fields_]
    return [{f: int(getattr(arr[k], f)) for f in names} for k in range(n)]


def _summary_from(s):
    return {f: int(getattr(s, f)) for f, _ in AetSummary._fields_}


def aet_get_event_log(h, raw: bool = False):
    """(events, summary); events as dicts, or the raw 64-byte records if raw."""
    lib = _lib.load()
    n = C.c_size_t()
    _check(h, lib.aet_get_event_log(h, None, 0, C.byref(n), None))
    arr = (AetEvent * max(1, n.value))()
    s = AetSummary()
    _check(h, lib.aet_get_event_log(h, arr, n.value, C.byref(n), C.byref(s)))
    if raw:
        return bytes(memoryview(arr))[:64 * n.value], _summary_from(s)
    return _events_from(arr, n.value), _summary_from(s)


def aet_debug_run_client_round(h, client: int, rnd: int, w_in, U_out=None, w_out=None, stream=None):
    P = aet_n_params(h)
    if U_out is None:
        U_out = np.empty(P, dtype=np.float32)
    if w_out is None:
        w_out = np.empty(P, dtype=np.float32)
    _check(h, _lib.load().aet_debug_run_client_round(h, client, rnd, _ptr(w_in), _ptr(U_out), _ptr(w_out),
                                                     _stream(stream)))
    return U_out, w_out


def aet_round_no_alloc(cfg, client: int, rnd: int, x, y, w_in, U_out, w_out, stream=None):
    """One round-task from caller-owned DEVICE buffers, using only the scratch
    array built into the library: for callers that may not allocate device
    memory while they run.  Asynchronous on the stream; calls that could overlap
    on the GPU race on the shared scratch."""
    conf = cfg if isinstance(cfg, AetConfig) else make_config(cfg)
    _check(None, _lib.load().aet_round_no_alloc(C.byref(conf), client, rnd, _ptr(x), _ptr(y), x.shape[0],
                                                _ptr(w_in), _ptr(U_out), _ptr(w_out), _stream(stream)))


def aet_debug_wait_probe(h, max_polls: int = 1 << 12, stream=None):
    """Makes a bounded device wait run out on purpose; raises AetError(AET_ERR_TIMEOUT)."""
    _check(h, _lib.load().aet_debug_wait_probe(h, max_polls, _stream(stream)))


def aet_set_kernel_timing(h, enable: bool):
    _check(h, _lib.load().aet_set_kernel_timing(h, int(enable)))


def aet_get_stats(h) -> dict:
    s = AetStats()
    _check(h, _lib.load().aet_get_stats(h, C.byref(s)))
    return dict(waves=int(s.waves), launches=[int(v) for v in s.launches],
                kernel_ms=[float(v) for v in s.kernel_ms], plan_ms=float(s.plan_ms))


def aet_schedule_only(cfg, n_rounds: int, raw: bool = False):
    """Host only: the event log a fresh run of n_rounds would produce."""
    lib = _lib.load()
    conf = cfg if isinstance(cfg, AetConfig) else make_config(cfg)
    n = C.c_size_t()
    _check(None, lib.aet_schedule_only(C.byref(conf), n_rounds, None, 0, C.byref(n), None))
    arr = (AetEvent * max(1, n.value))()
    s = AetSummary()
    _check(None, lib.aet_schedule_only(C.byref(conf), n_rounds, arr, n.value, C.byref(n), C.byref(s)))
    if raw:
        return bytes(memoryview(arr))[:64 * n.value], _summary_from(s)
    return _events_from(arr, n.value), _summary_from(s)


def aet_debug_draw(seed, stream_id, client, counter) -> int:
    return int(_lib.load().aet_debug_draw(seed, stream_id, client, counter))


def aet_debug_delay_ticks(dist, draw, p0, p1=0) -> int:
    return int(_lib.load().aet_debug_delay_ticks(dist, draw, p0, p1))


def aet_debug_plan_waves(cfg, n_rounds) -> int:
    conf = cfg if isinstance(cfg, AetConfig) else make_config(cfg)
    return int(_lib.load().aet_debug_plan_waves(C.byref(conf), n_rounds))


def aet_debug_plan_layout(cfg, n_rounds) -> dict:
    """Host only: the launch plan of a fresh run (see include/aet.h)."""
    conf = cfg if isinstance(cfg, AetConfig) else make_config(cfg)
    E = conf.n_clients * n_rounds
    u32 = lambda: np.zeros(max(E, 1), dtype=np.uint32)
    out = dict(task_seq=u32(), task_wave=u32(), task_snap_slot=u32(), u_row=u32(),
               snap_slot_after=np.zeros(max(E, 1), dtype=np.int32), apply_upto=u32())
    counts = np.zeros(3, dtype=np.uint32)
    _check(None, _lib.load().aet_debug_plan_layout(C.byref(conf), n_rounds, *[_ptr(v) for v in out.values()], _ptr(counts)))
    out = {k: v[:E] for k, v in out.items()}
    out["apply_upto"] = out["apply_upto"][:int(counts[0])]
    out.update(waves=int(counts[0]), n_u_rows=int(counts[1]), n_snap=int(counts[2]))
    return out


class Session:
    """Convenience wrapper: create, load every client's data, run, read back."""

    def __init__(self, cfg: dict, data, w0=None, stream=None):
        self.cfg = cfg
        self.h = aet_create(cfg)
        self.stream = stream
        try:
            if w0 is not None:
                aet_set_global_model(self.h, w0, stream)
            for c, (x, y) in enumerate(data):
                aet_load_client_data(self.h, c, x, y, stream)
        except Exception:
            self.close()
            raise

    def run(self, n_rounds=None):
        aet_run_rounds(self.h, self.cfg["n_rounds"] if n_rounds is None else n_rounds, self.stream)

    def reset(self):
        aet_reset(self.h, self.stream)

    def model(self):
        return aet_get_global_model(self.h, stream=self.stream)

    def log(self, raw=False):
        return aet_get_event_log(self.h, raw)

    def close(self):
        if self.h is not None:
            aet_destroy(self.h)
            self.h = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
