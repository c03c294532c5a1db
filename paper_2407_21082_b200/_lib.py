"""Loads libeexit.so and declares the C prototypes of include/eexit.h for ctypes."""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

_LIB = None

_p = C.c_void_p


class EEHead(C.Structure):
    """Mirror of `ee_head` in include/eexit.h."""
    _fields_ = [("h", _p), ("ld_h", C.c_longlong), ("gamma", _p), ("beta", _p), ("W", _p), ("tau_per_row", _p),
                ("tau", C.c_float), ("argmax", _p), ("entropy", _p), ("maxprob", _p), ("exit_mask", _p)]


EE_ROUND_MAX_DRAFT_HEADS = 8
HIDDEN_FN = C.CFUNCTYPE(C.c_int, _p, _p, C.c_int, C.c_int, _p, _p)


class EEDssdRoundArgs(C.Structure):
    """Mirror of `ee_dssd_round_args` in include/eexit.h."""
    _fields_ = [("S", C.c_int), ("k", C.c_int), ("d", C.c_int), ("V", C.c_int), ("ln_eps", C.c_float), ("eos_token", C.c_int),
                ("draft_head", EEHead), ("verify_head", EEHead), ("hidden", HIDDEN_FN), ("hidden_user", _p),
                ("last_tok", _p), ("out_tok", _p), ("capacity", C.c_int), ("seq_len", _p), ("finished", _p), ("stats", _p),
                ("draft_len", _p), ("accept_len", _p), ("next_tok", _p), ("workspace", _p), ("workspace_bytes", C.c_size_t),
                ("stream", _p), ("n_draft_heads", C.c_int), ("draft_heads", C.POINTER(EEHead)), ("head_use", _p),
                ("hidden_all_layers", C.c_int)]


EE_PLAN_MAX_HEADS = 16
EE_EXIT_HEAD_PLAN_BYTES = 64 + (EE_PLAN_MAX_HEADS // 4) * 2048


class EEExitHeadPlan(C.Structure):
    """Mirror of `ee_exit_head_plan` in include/eexit.h (opaque storage)."""
    _fields_ = [("opaque", C.c_ulonglong * (EE_EXIT_HEAD_PLAN_BYTES // 8))]


class EEHiddenTables(C.Structure):
    """Mirror of `ee_hidden_tables` in include/eexit.h."""
    _fields_ = [("table", _p * (EE_ROUND_MAX_DRAFT_HEADS + 1)), ("d", C.c_int), ("V", C.c_int), ("chained", C.c_int)]


PROTOTYPES = {
    "ee_status_string": (C.c_char_p, [C.c_int]),
    "ee_exit_head_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int]),
    "ee_exit_head_launches": (C.c_int, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "ee_workspace_init": (C.c_int, [_p, C.c_size_t, _p]),
    "ee_exit_head": (C.c_int, [_p, C.c_longlong, _p, _p, C.c_float, _p, C.c_int, C.c_int, C.c_int, _p, C.c_float,
                               _p, _p, _p, _p, _p, C.c_size_t, _p]),
    "ee_exit_head_top2": (C.c_int, [_p, C.c_longlong, _p, _p, C.c_float, _p, C.c_int, C.c_int, C.c_int, _p, C.c_float,
                                    _p, _p, _p, _p, _p, _p, C.c_size_t, _p]),
    "ee_exit_head_multi_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "ee_exit_head_multi_launches": (C.c_int, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "ee_exit_head_multi": (C.c_int, [C.POINTER(EEHead), C.c_int, C.c_float, C.c_int, C.c_int, C.c_int, _p, C.c_size_t, _p]),
    "ee_exit_head_plan_init": (C.c_int, [C.POINTER(EEExitHeadPlan), C.POINTER(EEHead), C.c_int, C.c_float, C.c_int, C.c_int, C.c_int,
                                         _p, C.c_size_t]),
    "ee_exit_head_plan_run": (C.c_int, [C.POINTER(EEExitHeadPlan), _p]),
    "ee_exit_head_plan_run_host": (C.c_int, [C.POINTER(EEExitHeadPlan), _p, _p, C.c_size_t, _p, _p, C.c_size_t, _p]),
    "ee_exit_head_path": (C.c_int, [_p, C.c_longlong, _p, _p, C.c_float, _p, C.c_int, C.c_int, C.c_int, _p, C.c_float,
                                    _p, _p, _p, _p, _p, C.c_size_t, _p, C.c_int]),
    "ee_exit_head_host": (C.c_int, [_p, _p, _p, _p, C.c_float, _p, C.c_int, C.c_int, C.c_int, _p, C.c_float,
                                    _p, _p, _p, _p, _p, _p, _p, _p, _p, C.c_size_t, _p]),
    "ee_exit_head_results_bytes": (C.c_size_t, [C.c_int, C.c_int]),
    "ee_exit_head_multi_host": (C.c_int, [C.POINTER(EEHead), C.c_int, C.c_float, C.c_int, C.c_int, C.c_int,
                                          _p, _p, _p, _p, _p, C.c_size_t, _p]),
    "ee_exit_head_static": (C.c_int, [_p, C.c_longlong, _p, _p, C.c_float, _p, C.c_int, C.c_int, C.c_int, _p, C.c_float,
                                      _p, _p, _p, _p, _p]),
    "ee_exit_head_static_query_error": (C.c_int, [_p]),
    "ee_exit_head_static_selftest_timeout": (C.c_int, [_p]),
    "ee_compact": (C.c_int, [_p, _p, C.c_longlong, C.c_int, C.c_int, _p, _p, _p, _p]),
    "dssd_accept": (C.c_int, [_p, _p, _p, C.c_int, C.c_int, C.c_int, _p, _p, _p, _p]),
    "dssd_commit": (C.c_int, [_p, _p, _p, C.c_int, C.c_int, C.c_int, C.c_int, _p, C.c_int, _p, _p, _p, _p, _p, _p, _p]),
    "dssd_round_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int]),
    "dssd_round_multi_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]),
    "dssd_round": (C.c_int, [C.POINTER(EEDssdRoundArgs)]),
    "ee_hidden_from_tables": (C.c_int, [_p, _p, C.c_int, C.c_int, _p, _p]),
    "ee_compact_accept": (C.c_int, [_p, _p, C.c_longlong, C.c_int, C.c_int, _p, _p, _p,
                                    _p, _p, _p, C.c_int, C.c_int, C.c_int, _p, _p, _p, _p]),
    "ee_head_kl_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int]),
    "ee_head_kl": (C.c_int, [_p, C.c_longlong, _p, _p, _p, _p, C.c_longlong, _p, _p, _p, C.c_float, C.c_int, C.c_int, C.c_int,
                             _p, _p, _p, _p, _p, C.c_size_t, _p]),
    "ee_cascade_workspace_bytes": (C.c_size_t, [C.c_int, C.c_int, C.c_int]),
    "ee_cascade": (C.c_int, [C.POINTER(EEHead), C.c_int, C.c_float, C.c_int, C.c_int, C.c_int, _p, _p, _p, _p,
                             _p, C.c_size_t, _p]),
    "ee_calibrate_workspace_bytes": (C.c_size_t, [C.c_int]),
    "ee_calibrate": (C.c_int, [_p, _p, _p, C.c_int, C.c_double, _p, _p, _p, C.c_size_t, _p]),
    "ee_query_async_error": (C.c_int, [_p, _p]),
    "ee_selftest_wait_timeout": (C.c_int, [_p, C.c_size_t, _p]),
    "ee_selftest_read_stream": (C.c_int, [_p, C.c_size_t, _p, C.c_size_t, _p]),
}


def lib_path() -> str:
    return _build.LIB


def load() -> C.CDLL:
    """Returns the loaded library.  Raises if it has not been built: there is no fallback path."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2407_21082_b200.build` "
                               "(needs nvcc); this package has no other implementation")
        lib = C.CDLL(path)
        for name, (res, args) in PROTOTYPES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _LIB = lib
    return _LIB
