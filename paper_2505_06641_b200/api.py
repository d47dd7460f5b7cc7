"""Thin Python binding of the C ABI in ``include/sneakpeek.h`` (argument marshalling only).

Every function has the name and the argument order of its C counterpart; tensors are passed as
``torch.Tensor`` (device arguments) or ``numpy.ndarray`` (host arguments) and only their data pointers
cross the boundary.  Nothing is computed here, and there is no fallback: if ``libsneakpeek.so`` has not
been built (``python -m paper_2505_06641_b200.build``) importing the library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

from .build import LIB_PATH

SP_OK, SP_EINVAL, SP_ENOMEM, SP_ECUDA, SP_ESTATE, SP_ELIMIT = range(6)
SP_F32, SP_BF16 = 0, 1
SP_PENDING, SP_SCHEDULED, SP_EXPIRED = 0, 1, 2
_STATUS_NAMES = ["SP_OK", "SP_EINVAL", "SP_ENOMEM", "SP_ECUDA", "SP_ESTATE", "SP_ELIMIT"]

ROUND_DTYPE = np.dtype([
    ("instance", "<i4"), ("round", "<i4"), ("app", "<i4"), ("model", "<i4"), ("batch", "<i4"),
    ("n_members", "<i4"), ("n_expired", "<i4"), ("exact", "<i4"), ("t_start_ns", "<i8"), ("t_end_ns", "<i8"),
    ("utility", "<f8"), ("group_priority", "<f8")], align=True)
REQ_DTYPE = np.dtype([("status", "<i4"), ("round", "<i4"), ("model", "<i4"), ("worker", "<i4"), ("order", "<i8")],
                     align=True)
assert ROUND_DTYPE.itemsize == 64 and REQ_DTYPE.itemsize == 24

EXPORTS = ["sp_create", "sp_destroy", "sp_last_error", "sp_load_profiles", "sp_default_options", "sp_set_options", "sp_set_clock",
           "sp_set_clocks", "sp_score", "sp_get_scores", "sp_schedule_round", "sp_get_requests", "sp_get_clocks",
           "sp_reset", "sp_check", "sp_get_stats", "sp_run_host", "sp_score_static", "sp_schedule_split",
           "sp_schedule_exhaustive", "sp_schedule_baseline", "sp_get_labels", "sp_set_workers", "sp_schedule_workers",
           "sp_get_workers", "sp_load_evidence", "sp_score_knn"]
SP_BASE_MAXACC_EDF, SP_BASE_LO_EDF, SP_BASE_LO_PRIORITY = 0, 1, 2


class SpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (_STATUS_NAMES[status] if 0 <= status < 6 else status, message))
        self.status = status


class _Profiles(C.Structure):
    _fields_ = [
        ("n_instances", C.c_int32), ("n_apps", C.c_int32), ("n_classes", C.c_int32), ("feat_dim", C.c_int32),
        ("feat_dtype", C.c_int32), ("models_per_app", C.c_void_p), ("head_w", C.c_void_p), ("head_b", C.c_void_p),
        ("prior_alpha", C.c_void_p), ("evidence_k", C.c_float), ("recall", C.c_void_p),
        ("lat_alpha_ns", C.c_void_p), ("lat_beta_ns", C.c_void_p), ("swap_ns", C.c_void_p),
        ("batch_sizes", C.c_void_p), ("n_batch_sizes", C.c_int32), ("penalty_kind", C.c_void_p),
        ("prio_time_scale_s", C.c_double)]


class _Options(C.Structure):
    _fields_ = [("trace_mode", C.c_int32), ("timing", C.c_int32), ("guard_utility", C.c_double),
                ("guard_priority", C.c_double)]


class _Stats(C.Structure):
    _fields_ = [("kernel_launches", C.c_int64), ("rounds", C.c_int64), ("exact_utility", C.c_int64),
                ("exact_priority", C.c_int64), ("exact_rows", C.c_int64), ("score_calls", C.c_int64),
                ("sched_calls", C.c_int64), ("score_kernel_ms", C.c_double), ("sched_kernel_ms", C.c_double),
                ("score_kernel", C.c_int32), ("pad_", C.c_int32)]


class _StaticHead(C.Structure):
    _fields_ = [("n_apps", C.c_int32), ("n_classes", C.c_int32), ("feat_dim", C.c_int32), ("feat_dtype", C.c_int32),
                ("models_per_app", C.c_void_p), ("head_w", C.c_void_p), ("head_b", C.c_void_p), ("recall", C.c_void_p)]


class _KnnEvidence(C.Structure):
    _fields_ = [("k", C.c_int32), ("n_ref", C.c_int64), ("ref_feats", C.c_void_p), ("ref_label", C.c_void_p),
                ("ref_app", C.c_void_p)]


_lib = None


def load_library():
    """Loads ``libsneakpeek.so``; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("CUDA library %s is missing: build it with `python -m paper_2505_06641_b200.build` "
                           "(there is no CPU fallback)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.sp_create.argtypes = [C.POINTER(vp), C.c_int, vp]
    lib.sp_destroy.argtypes = [vp]
    lib.sp_destroy.restype = None
    lib.sp_last_error.argtypes = [vp]
    lib.sp_last_error.restype = C.c_char_p
    lib.sp_load_profiles.argtypes = [vp, C.POINTER(_Profiles)]
    lib.sp_set_options.argtypes = [vp, C.POINTER(_Options)]
    lib.sp_default_options.argtypes = [C.POINTER(_Options)]
    lib.sp_default_options.restype = None
    lib.sp_set_clock.argtypes = [vp, i32, i64, i32]
    lib.sp_set_clocks.argtypes = [vp, vp, vp]
    lib.sp_score.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp]
    lib.sp_get_scores.argtypes = [vp, i64, i64, vp, vp]
    lib.sp_schedule_round.argtypes = [vp, i32, vp, i64, vp]
    lib.sp_get_requests.argtypes = [vp, i64, i64, vp]
    lib.sp_get_clocks.argtypes = [vp, vp, vp]
    lib.sp_reset.argtypes = [vp]
    lib.sp_check.argtypes = [vp]
    lib.sp_get_stats.argtypes = [vp, C.POINTER(_Stats)]
    lib.sp_run_host.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, i64, vp]
    lib.sp_schedule_split.argtypes = [vp, vp, i64, vp]
    lib.sp_schedule_exhaustive.argtypes = [vp, i32, vp, i64, vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    lib.sp_schedule_baseline.argtypes = [vp, i32, vp, i64, vp]
    lib.sp_get_labels.argtypes = [vp, i64, i64, vp]
    lib.sp_load_evidence.argtypes = [vp, C.POINTER(_KnnEvidence)]
    lib.sp_score_knn.argtypes = [vp, i64, vp, vp, vp, vp, vp]
    lib.sp_set_workers.argtypes = [vp, i32, vp, vp, vp]
    lib.sp_schedule_workers.argtypes = [vp, i32, vp, i64, vp]
    lib.sp_get_workers.argtypes = [vp, vp, vp]
    lib.sp_score_static.argtypes = [C.c_int, vp, C.POINTER(_StaticHead), i64, vp, vp, vp, vp, C.c_char_p, i32]
    for name in EXPORTS:
        if name not in ("sp_destroy", "sp_last_error", "sp_default_options"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _dev(t) -> Optional[int]:
    """Device pointer of a torch tensor (None stays NULL)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _host(a: Optional[np.ndarray]) -> Optional[int]:
    if a is None:
        return None
    if not a.flags["C_CONTIGUOUS"]:
        raise ValueError("expected a C-contiguous array")
    return a.ctypes.data


def _ok(ctx, status: int):
    if status != SP_OK:
        raise SpError(status, sp_last_error(ctx))


# ---------------------------------------------------------------------------------------------- C ABI, 1:1

def sp_create(device: int = 0, cuda_stream: int = 0) -> int:
    out = C.c_void_p()
    st = load_library().sp_create(C.byref(out), int(device), C.c_void_p(cuda_stream or None))
    if st != SP_OK or not out.value:
        raise SpError(st, "sp_create failed (no usable CUDA device?)")
    return out.value


def sp_destroy(ctx: int) -> None:
    load_library().sp_destroy(ctx)


def sp_last_error(ctx: int) -> str:
    return load_library().sp_last_error(ctx).decode()


def sp_load_profiles(ctx: int, w) -> None:
    """``w``: any object with the profile fields of ``synth.Workload`` (numpy arrays, host memory)."""
    f = lambda a, dt: np.ascontiguousarray(a, dtype=dt)
    wdt = np.uint16 if int(w.feat_dtype) == SP_BF16 else np.float32
    keep = dict(mpa=f(w.models_per_app, np.int32), head_w=f(w.head_w, wdt), head_b=f(w.head_b, np.float32),
                prior=None if w.prior_alpha is None else f(w.prior_alpha, np.float32),
                recall=f(w.recall, np.float32), al=f(w.lat_alpha_ns, np.int64), be=f(w.lat_beta_ns, np.int64),
                sw=f(w.swap_ns, np.int64), bs=f(w.batch_sizes, np.int32),
                pen=None if getattr(w, "penalty_kind", None) is None else f(w.penalty_kind, np.int32))
    p = _Profiles(int(w.n_instances), int(w.n_apps), int(w.n_classes), int(w.feat_dim), int(w.feat_dtype),
                  _host(keep["mpa"]), _host(keep["head_w"]), _host(keep["head_b"]), _host(keep["prior"]),
                  float(w.evidence_k), _host(keep["recall"]), _host(keep["al"]), _host(keep["be"]), _host(keep["sw"]),
                  _host(keep["bs"]), int(keep["bs"].shape[0]), _host(keep["pen"]), float(w.prio_time_scale_s))
    _ok(ctx, load_library().sp_load_profiles(ctx, C.byref(p)))


def sp_default_options() -> dict:
    o = _Options()
    load_library().sp_default_options(C.byref(o))
    return {k: getattr(o, k) for k, _ in _Options._fields_}


def sp_set_options(ctx: int, trace_mode: bool = False, guard_utility: float = 2e-5,
                   guard_priority: float = 2e-6, timing: bool = False) -> None:
    o = _Options(int(bool(trace_mode)), int(bool(timing)), float(guard_utility), float(guard_priority))
    _ok(ctx, load_library().sp_set_options(ctx, C.byref(o)))


def sp_set_clock(ctx: int, instance: int, t_ns: int, loaded_model: int) -> None:
    _ok(ctx, load_library().sp_set_clock(ctx, int(instance), int(t_ns), int(loaded_model)))


def sp_set_clocks(ctx: int, t_ns=None, loaded_model=None) -> None:
    _ok(ctx, load_library().sp_set_clocks(ctx, _dev(t_ns), _dev(loaded_model)))


def sp_score(ctx: int, n: int, feats, app, arrival_ns, deadline_ns, instance=None, acc_out=None) -> None:
    _ok(ctx, load_library().sp_score(ctx, int(n), _dev(feats), _dev(app), _dev(arrival_ns), _dev(deadline_ns),
                                     _dev(instance), _dev(acc_out)))


def sp_load_evidence(ctx: int, k: int, ref_feats: np.ndarray, ref_label: np.ndarray, ref_app: np.ndarray) -> None:
    """Reference set of the k-nearest-neighbour SneakPeek model (host arrays; bf16 features as uint16 bit patterns)."""
    rf = np.ascontiguousarray(ref_feats)
    rl, ra = np.ascontiguousarray(ref_label, dtype=np.int32), np.ascontiguousarray(ref_app, dtype=np.int32)
    ev = _KnnEvidence(int(k), int(rf.shape[0]), _host(rf), _host(rl), _host(ra))
    _ok(ctx, load_library().sp_load_evidence(ctx, C.byref(ev)))


def sp_score_knn(ctx: int, n: int, feats, app, arrival_ns, deadline_ns, acc_out=None) -> None:
    _ok(ctx, load_library().sp_score_knn(ctx, int(n), _dev(feats), _dev(app), _dev(arrival_ns), _dev(deadline_ns),
                                         _dev(acc_out)))


def sp_get_scores(ctx: int, first: int, n: int, acc=None, v=None) -> None:
    _ok(ctx, load_library().sp_get_scores(ctx, int(first), int(n), _dev(acc), _dev(v)))


def sp_schedule_round(ctx: int, max_rounds: int, rounds_out=None, cap: int = 0, n_done=None) -> None:
    _ok(ctx, load_library().sp_schedule_round(ctx, int(max_rounds), _dev(rounds_out), int(cap), _dev(n_done)))


def sp_schedule_split(ctx: int, rounds_out=None, cap: int = 0, n_done=None) -> None:
    _ok(ctx, load_library().sp_schedule_split(ctx, _dev(rounds_out), int(cap), _dev(n_done)))


def sp_schedule_exhaustive(ctx: int, split: bool, rounds_out=None, cap: int = 0, n_done=None):
    """Returns (best total utility, number of solutions visited)."""
    total, nsol = C.c_double(), C.c_int64()
    _ok(ctx, load_library().sp_schedule_exhaustive(ctx, int(bool(split)), _dev(rounds_out), int(cap), _dev(n_done),
                                                   C.byref(total), C.byref(nsol)))
    return total.value, nsol.value


def sp_schedule_baseline(ctx: int, policy: int, rounds_out=None, cap: int = 0, n_done=None) -> None:
    _ok(ctx, load_library().sp_schedule_baseline(ctx, int(policy), _dev(rounds_out), int(cap), _dev(n_done)))


def sp_set_workers(ctx: int, lat_alpha_ns: np.ndarray, lat_beta_ns: np.ndarray, swap_ns: np.ndarray) -> None:
    """Registers W workers; the three arrays are host arrays [W, sumM] of int64 nanoseconds."""
    al, be, sw = (np.ascontiguousarray(a, dtype=np.int64) for a in (lat_alpha_ns, lat_beta_ns, swap_ns))
    _ok(ctx, load_library().sp_set_workers(ctx, int(al.shape[0]), _host(al), _host(be), _host(sw)))


def sp_schedule_workers(ctx: int, split: bool, rounds_out=None, cap: int = 0, n_done=None) -> None:
    _ok(ctx, load_library().sp_schedule_workers(ctx, int(bool(split)), _dev(rounds_out), int(cap), _dev(n_done)))


def sp_get_workers(ctx: int, t_ns=None, loaded=None) -> None:
    _ok(ctx, load_library().sp_get_workers(ctx, _dev(t_ns), _dev(loaded)))


def sp_get_labels(ctx: int, first: int, n: int, labels) -> None:
    _ok(ctx, load_library().sp_get_labels(ctx, int(first), int(n), _dev(labels)))


def sp_get_requests(ctx: int, first: int, n: int, out) -> None:
    _ok(ctx, load_library().sp_get_requests(ctx, int(first), int(n), _dev(out)))


def sp_get_clocks(ctx: int, t_ns=None, loaded_model=None) -> None:
    _ok(ctx, load_library().sp_get_clocks(ctx, _dev(t_ns), _dev(loaded_model)))


def sp_reset(ctx: int) -> None:
    _ok(ctx, load_library().sp_reset(ctx))


def sp_check(ctx: int) -> None:
    _ok(ctx, load_library().sp_check(ctx))


def sp_get_stats(ctx: int) -> dict:
    s = _Stats()
    _ok(ctx, load_library().sp_get_stats(ctx, C.byref(s)))
    return {k: getattr(s, k) for k, _ in _Stats._fields_}


def sp_run_host(ctx: int, n: int, feats: np.ndarray, app: np.ndarray, arrival_ns: np.ndarray,
                deadline_ns: np.ndarray, instance: Optional[np.ndarray], t0_ns: Optional[np.ndarray],
                loaded0: Optional[np.ndarray], max_rounds: int, reqs_out: Optional[np.ndarray] = None,
                rounds_out: Optional[np.ndarray] = None, cap: int = 0, n_done: Optional[np.ndarray] = None) -> None:
    _ok(ctx, load_library().sp_run_host(ctx, int(n), _host(feats), _host(app), _host(arrival_ns), _host(deadline_ns),
                                        _host(instance), _host(t0_ns), _host(loaded0), int(max_rounds),
                                        _host(reqs_out), _host(rounds_out), int(cap), _host(n_done)))


def sp_score_static(device: int, cuda_stream: int, n_apps: int, n_classes: int, feat_dim: int, feat_dtype: int,
                    models_per_app: np.ndarray, head_w, head_b, recall, n: int, feats, app, acc_out, v_out) -> None:
    """Allocation-free scoring of one instance: device tensors in, device tensors out, fixed built-in scratch.

    ``models_per_app`` is a host array; ``head_w``, ``head_b``, ``recall``, ``feats``, ``app`` and the two outputs
    are CUDA tensors.  Raises ``SpError`` (with the library's message) on bad arguments, e.g. n > 65,536.
    """
    mpa = np.ascontiguousarray(models_per_app, dtype=np.int32)
    head = _StaticHead(int(n_apps), int(n_classes), int(feat_dim), int(feat_dtype), _host(mpa), _dev(head_w),
                       _dev(head_b), _dev(recall))
    err = C.create_string_buffer(256)
    st = load_library().sp_score_static(int(device), C.c_void_p(cuda_stream or None), C.byref(head), int(n),
                                        _dev(feats), _dev(app), _dev(acc_out), _dev(v_out), err, 256)
    if st != SP_OK:
        raise SpError(st, err.value.decode())
