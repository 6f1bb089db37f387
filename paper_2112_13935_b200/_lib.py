"""ctypes view of libaet_b200.so: structs, prototypes, loader.

Argument marshalling only.  The library is built in-tree by ``build.py``; if it
is missing the import of this module fails loudly - there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libaet_b200.so")

NEVER_WAIT = 0xFFFFFFFF
STATUS_NAMES = ["AET_OK", "AET_ERR_ARG", "AET_ERR_CONFIG", "AET_ERR_STATE", "AET_ERR_NOMEM",
                "AET_ERR_CUDA", "AET_ERR_TIMEOUT", "AET_ERR_NUMERIC"]


class AetConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("n_clients", C.c_uint32), ("model", C.c_uint32),
        ("n_layers", C.c_uint32), ("dims", C.c_uint32 * 8), ("precision", C.c_uint32),
        ("batch", C.c_uint32), ("sched_a", C.c_uint32), ("sched_b", C.c_uint32),
        ("round_base", C.c_uint32), ("max_lag_d", C.c_uint32), ("lr", C.c_float),
        ("lr_beta", C.c_float), ("l2", C.c_float), ("delay_dist", C.c_uint32),
        ("seed", C.c_uint64), ("compute_delay_mean", C.c_double), ("network_delay_mean", C.c_double),
        ("compute_delay_lo", C.c_double), ("compute_delay_hi", C.c_double),
        ("network_delay_lo", C.c_double), ("network_delay_hi", C.c_double),
        ("straggler_factor", C.c_double), ("n_stragglers", C.c_uint32), ("flags", C.c_uint32),
        ("split_mode", C.c_uint32), ("topology", C.c_uint32), ("client_shares", C.POINTER(C.c_uint32)),
    ]


class AetEvent(C.Structure):
    _fields_ = [
        ("t_start", C.c_uint64), ("t_trigger", C.c_uint64), ("t_apply", C.c_uint64),
        ("wait_ticks", C.c_uint64), ("client", C.c_uint32), ("round", C.c_uint32),
        ("samples", C.c_uint32), ("steps", C.c_uint32), ("seq", C.c_uint32),
        ("seen", C.c_uint32), ("lag", C.c_uint32), ("dest", C.c_uint32),
    ]


class AetSummary(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("messages_up", "model_pulls", "samples_total",
                                          "messages_if_per_sample", "messages_if_constant_b",
                                          "t_end_ticks")]


class AetStats(C.Structure):
    _fields_ = [("waves", C.c_uint64), ("launches", C.c_uint64 * 4), ("kernel_ms", C.c_double * 4),
                ("plan_ms", C.c_double)]


# name -> (restype, argtypes); every symbol include/aet.h declares
PROTOTYPES = {
    "aet_create": (C.c_int, [C.POINTER(AetConfig), C.POINTER(C.c_void_p)]),
    "aet_destroy": (C.c_int, [C.c_void_p]),
    "aet_reset": (C.c_int, [C.c_void_p, C.c_void_p]),
    "aet_set_global_model": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "aet_load_client_data": (C.c_int, [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]),
    "aet_prepare_rounds": (C.c_int, [C.c_void_p, C.c_uint32]),
    "aet_run_rounds": (C.c_int, [C.c_void_p, C.c_uint32, C.c_void_p]),
    "aet_get_global_model": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "aet_get_node_model": (C.c_int, [C.c_void_p, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "aet_get_event_log": (C.c_int, [C.c_void_p, C.POINTER(AetEvent), C.c_size_t, C.POINTER(C.c_size_t),
                                    C.POINTER(AetSummary)]),
    "aet_get_update_sum": (C.c_int, [C.c_void_p, C.c_uint32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "aet_debug_run_client_round": (C.c_int, [C.c_void_p, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_void_p]),
    "aet_debug_wait_probe": (C.c_int, [C.c_void_p, C.c_uint32, C.c_void_p]),
    "aet_set_kernel_timing": (C.c_int, [C.c_void_p, C.c_int]),
    "aet_get_stats": (C.c_int, [C.c_void_p, C.POINTER(AetStats)]),
    "aet_n_params": (C.c_size_t, [C.c_void_p]),
    "aet_last_error": (C.c_char_p, [C.c_void_p]),
    "aet_round_no_alloc": (C.c_int, [C.POINTER(AetConfig), C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p,
                                     C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "aet_schedule_only": (C.c_int, [C.POINTER(AetConfig), C.c_uint32, C.POINTER(AetEvent), C.c_size_t,
                                    C.POINTER(C.c_size_t), C.POINTER(AetSummary)]),
    "aet_debug_draw": (C.c_uint64, [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]),
    "aet_debug_delay_ticks": (C.c_uint64, [C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64]),
    "aet_debug_plan_waves": (C.c_uint32, [C.POINTER(AetConfig), C.c_uint32]),
    "aet_debug_plan_layout": (C.c_int, [C.POINTER(AetConfig), C.c_uint32] + [C.c_void_p] * 7),
}

_lib = None


def load():
    """The loaded library with prototypes set.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2112_13935_b200.build` "
            "(needs nvcc).  There is no CPU fallback.")
    lib = C.CDLL(LIB_PATH)
    for name, (res, args) in PROTOTYPES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib
