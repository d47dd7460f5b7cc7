"""ctypes front end of the CPU oracle (test infrastructure, not the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.  It
compiles ``sneakpeek_oracle.c`` with gcc on first use and exposes two calls that take the same
arrays the CUDA library takes:

* :func:`score`  -- data-aware accuracy ``acc[n, Mmax]`` (Eq. 9 of the paper over the Dirichlet
  posterior mean of Eq. 10-11) and the priority factor ``v[n] = 1 + Var`` (Eq. 12), in fp64;
* :func:`drain`  -- the greedy group-level rounds (Eq. 13-14, Algorithm 1) until nothing is left, over whole
  applications or over the data-aware sub-groups of Section 4.3 (``labels=``);
* :func:`bruteforce` -- Algorithm 1's exhaustive branch over the groups of one instance;
* :func:`baseline` -- the request-level baselines of Section 5.1 (MaxAcc-EDF, LO-EDF, LO-Priority).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sneakpeek_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, no FMA contraction, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Profiles(C.Structure):
    _fields_ = [
        ("n_instances", C.c_int32), ("n_apps", C.c_int32), ("n_classes", C.c_int32),
        ("feat_dim", C.c_int32), ("feat_dtype", C.c_int32),
        ("models_per_app", C.c_void_p), ("head_w", C.c_void_p), ("head_b", C.c_void_p),
        ("prior_alpha", C.c_void_p), ("evidence_k", C.c_double), ("recall", C.c_void_p),
        ("lat_alpha_ns", C.c_void_p), ("lat_beta_ns", C.c_void_p), ("swap_ns", C.c_void_p),
        ("batch_sizes", C.c_void_p), ("n_batch_sizes", C.c_int32),
        ("prio_time_scale_s", C.c_double), ("penalty_kind", C.c_void_p),
    ]


ROUND_DTYPE = np.dtype([
    ("instance", "<i4"), ("round", "<i4"), ("app", "<i4"), ("model", "<i4"), ("batch", "<i4"),
    ("n_members", "<i4"), ("n_expired", "<i4"), ("label", "<i4"), ("worker", "<i4"), ("pad_", "<i4"), ("t_start_ns", "<i8"),
    ("t_end_ns", "<i8"), ("utility", "<f8"), ("group_priority", "<f8"), ("util_margin", "<f8"),
    ("prio_margin", "<f8")], align=True)
REQ_DTYPE = np.dtype([("status", "<i4"), ("round", "<i4"), ("model", "<i4"), ("worker", "<i4"),
                      ("order", "<i8")], align=True)

PENDING, SCHEDULED, EXPIRED = 0, 1, 2


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.orc_score.restype = C.c_int
        lib.orc_score.argtypes = [C.POINTER(_Profiles), C.c_int64] + [C.c_void_p] * 7
        lib.orc_drain.restype = C.c_int
        lib.orc_drain.argtypes = ([C.POINTER(_Profiles), C.c_int64] + [C.c_void_p] * 9 +
                                  [C.c_int, C.c_int64, C.c_void_p, C.c_int64] + [C.c_void_p] * 4)
        lib.orc_bruteforce.restype = C.c_int
        lib.orc_bruteforce.argtypes = ([C.POINTER(_Profiles), C.c_int64] + [C.c_void_p] * 5 + [C.c_int64, C.c_int32,
                                       C.c_void_p, C.c_int64] + [C.c_void_p] * 7)
        lib.orc_drain_workers.restype = C.c_int
        lib.orc_drain_workers.argtypes = ([C.POINTER(_Profiles), C.c_int, C.c_int64] + [C.c_void_p] * 6 +
                                          [C.c_int64, C.c_int32, C.c_int, C.c_int64, C.c_void_p, C.c_int64] + [C.c_void_p] * 4)
        lib.orc_score_knn.restype = C.c_int
        lib.orc_score_knn.argtypes = ([C.POINTER(_Profiles), C.c_int, C.c_int64] + [C.c_void_p] * 3 + [C.c_int64] +
                                      [C.c_void_p] * 6)
        lib.orc_baseline.restype = C.c_int
        lib.orc_baseline.argtypes = ([C.POINTER(_Profiles), C.c_int, C.c_int64] + [C.c_void_p] * 9 +
                                     [C.c_int64] + [C.c_void_p] * 5)
        lib.orc_num_threads.restype = C.c_int
        lib.orc_penalty.restype = C.c_double
        lib.orc_penalty.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def penalty(kind: int, deadline_ns: int, arrival_ns: int, completion_ns: int) -> float:
    """gamma of Eq. 2 under the stated reading of Section 5.1 (0 step, 1 linear, 2 sigmoid)."""
    return float(_load().orc_penalty(int(kind), int(deadline_ns), int(arrival_ns), int(completion_ns)))


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


class _Bound:
    """Keeps contiguous copies of the profile arrays alive next to the C struct."""

    def __init__(self, w):
        f = lambda a, dt: np.ascontiguousarray(a, dtype=dt)
        wdt = np.uint16 if w.feat_dtype == 1 else np.float32
        self.keep = dict(
            mpa=f(w.models_per_app, np.int32), head_w=f(w.head_w, wdt), head_b=f(w.head_b, np.float32),
            prior=None if w.prior_alpha is None else f(w.prior_alpha, np.float32),
            recall=f(w.recall, np.float32), al=f(w.lat_alpha_ns, np.int64), be=f(w.lat_beta_ns, np.int64),
            sw=f(w.swap_ns, np.int64), bs=f(w.batch_sizes, np.int32),
            pen=f(w.penalty_kind, np.int32))
        k = self.keep
        self.struct = _Profiles(
            int(w.n_instances), int(w.n_apps), int(w.n_classes), int(w.feat_dim), int(w.feat_dtype),
            _ptr(k["mpa"]), _ptr(k["head_w"]), _ptr(k["head_b"]), _ptr(k["prior"]), float(np.float32(w.evidence_k)),   # the interface takes kappa as a float
            _ptr(k["recall"]), _ptr(k["al"]), _ptr(k["be"]), _ptr(k["sw"]), _ptr(k["bs"]),
            int(k["bs"].shape[0]), float(w.prio_time_scale_s), _ptr(k["pen"]))


@dataclass
class Scores:
    acc: np.ndarray      # [n, Mmax] float64
    v: np.ndarray        # [n] float64
    theta: Optional[np.ndarray]  # [n, C] float64 when requested
    label: Optional[np.ndarray] = None  # [n] int32: label c with theta_c > 0.5, -1 when there is none


def score(w, want_theta: bool = False) -> Scores:
    """Steps a1-a4 for every request of workload ``w`` (any object with the Workload fields)."""
    lib, b = _load(), _Bound(w)
    n = int(w.app.shape[0])
    mm = int(np.max(w.models_per_app))
    fdt = np.uint16 if w.feat_dtype == 1 else np.float32
    feats = np.ascontiguousarray(w.feats, dtype=fdt)
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    inst = np.ascontiguousarray(w.instance, dtype=np.int32)
    acc = np.zeros((n, mm), dtype=np.float64)
    v = np.zeros(n, dtype=np.float64)
    theta = np.zeros((n, int(w.n_classes)), dtype=np.float64) if want_theta else None
    label = np.zeros(n, dtype=np.int32)
    rc = lib.orc_score(C.byref(b.struct), n, _ptr(feats), _ptr(app), _ptr(inst), _ptr(acc), _ptr(v), _ptr(theta), _ptr(label))
    if rc != 0:
        raise ValueError("orc_score rejected its arguments")
    return Scores(acc, v, theta, label)


@dataclass
class Drain:
    rounds: np.ndarray      # [I, cap] ROUND_DTYPE (entries >= n_rounds[i] are zero)
    n_rounds: np.ndarray    # [I] int64
    reqs: np.ndarray        # [n] REQ_DTYPE
    t_end_ns: np.ndarray    # [I] int64
    loaded_end: np.ndarray  # [I] int32


def drain(w, acc: np.ndarray, v: np.ndarray, t0_ns=None, loaded0=None, max_rounds: Optional[int] = None,
          cap: Optional[int] = None, trace_mode: Optional[bool] = None, labels: Optional[np.ndarray] = None) -> Drain:
    """Runs the rounds of every instance of ``w`` from clock ``t0_ns`` with model ``loaded0`` resident.

    ``labels`` (from :func:`score`) switches to the data-aware sub-groups of Section 4.3: requests of an application
    with the same predicted label form a group of their own."""
    lib, b = _load(), _Bound(w)
    n, ni = int(w.app.shape[0]), int(w.n_instances)
    per_inst = int(np.max(np.bincount(np.asarray(w.instance), minlength=ni))) if n else 0
    if max_rounds is None:
        max_rounds = per_inst + 1
    if cap is None:
        cap = max(1, min(max_rounds, per_inst))
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    inst = np.ascontiguousarray(w.instance, dtype=np.int32)
    arr = np.ascontiguousarray(w.arrival_ns, dtype=np.int64)
    dl = np.ascontiguousarray(w.deadline_ns, dtype=np.int64)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    t0 = np.ascontiguousarray(w.t0_ns if t0_ns is None else t0_ns, dtype=np.int64)
    l0 = np.full(ni, -1, dtype=np.int32) if loaded0 is None else np.ascontiguousarray(loaded0, dtype=np.int32)
    rounds = np.zeros((ni, cap), dtype=ROUND_DTYPE)
    n_rounds = np.zeros(ni, dtype=np.int64)
    reqs = np.zeros(n, dtype=REQ_DTYPE)
    t_end = np.zeros(ni, dtype=np.int64)
    l_end = np.zeros(ni, dtype=np.int32)
    tm = bool(w.trace_mode) if trace_mode is None else bool(trace_mode)
    lab = None if labels is None else np.ascontiguousarray(labels, dtype=np.int32)
    rc = lib.orc_drain(C.byref(b.struct), n, _ptr(app), _ptr(inst), _ptr(lab), _ptr(arr), _ptr(dl), _ptr(acc), _ptr(v),
                       _ptr(t0), _ptr(l0), int(tm), int(max_rounds), _ptr(rounds), int(cap), _ptr(n_rounds),
                       _ptr(reqs), _ptr(t_end), _ptr(l_end))
    if rc != 0:
        raise ValueError("orc_drain rejected its arguments")
    return Drain(rounds, n_rounds, reqs, t_end, l_end)


@dataclass
class BruteForce:
    rounds: np.ndarray      # [1, cap] ROUND_DTYPE, one record per executed batch
    n_rounds: np.ndarray    # [1]
    reqs: np.ndarray        # [n] REQ_DTYPE
    t_end_ns: np.ndarray    # [1]
    loaded_end: np.ndarray  # [1]
    total: float            # best total utility (the sum inside Eq. 3)
    second: float           # best total among the solutions with a different total (-inf if none)
    n_solutions: int        # solutions visited = G! * prod M_g


def bruteforce(w, acc: np.ndarray, labels: Optional[np.ndarray] = None, loaded0: int = -1) -> BruteForce:
    """Exact group-level solution of a single-instance workload (Algorithm 1's branch for few groups)."""
    lib, b = _load(), _Bound(w)
    if int(w.n_instances) != 1:
        raise ValueError("one instance only")
    n = int(w.app.shape[0])
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    arr = np.ascontiguousarray(w.arrival_ns, dtype=np.int64)
    dl = np.ascontiguousarray(w.deadline_ns, dtype=np.int64)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    lab = None if labels is None else np.ascontiguousarray(labels, dtype=np.int32)
    cap = max(1, n)
    rounds = np.zeros((1, cap), dtype=ROUND_DTYPE)
    n_rounds = np.zeros(1, dtype=np.int64)
    reqs = np.zeros(n, dtype=REQ_DTYPE)
    t_end = np.zeros(1, dtype=np.int64)
    l_end = np.zeros(1, dtype=np.int32)
    best, second, nsol = np.zeros(1), np.zeros(1), np.zeros(1, dtype=np.int64)
    rc = lib.orc_bruteforce(C.byref(b.struct), n, _ptr(app), _ptr(lab), _ptr(arr), _ptr(dl), _ptr(acc), int(w.t0_ns[0]),
                            int(loaded0), _ptr(rounds), cap, _ptr(n_rounds), _ptr(reqs), _ptr(t_end), _ptr(l_end),
                            _ptr(best), _ptr(second), _ptr(nsol))
    if rc != 0:
        raise ValueError("orc_bruteforce: %s" % ("too many groups or solutions" if rc == -2 else "bad arguments"))
    return BruteForce(rounds, n_rounds, reqs, t_end, l_end, float(best[0]), float(second[0]), int(nsol[0]))


MAXACC_EDF, LO_EDF, LO_PRIORITY = 0, 1, 2


@dataclass
class Baseline:
    rounds: np.ndarray      # [I, cap] ROUND_DTYPE, one record per request in execution order
    n_rounds: np.ndarray    # [I]
    reqs: np.ndarray        # [n] REQ_DTYPE
    t_end_ns: np.ndarray    # [I]
    loaded_end: np.ndarray  # [I]
    min_margin: np.ndarray  # [I] smallest relative gap between the two best scores of a decision / two neighbours of the order


def baseline(w, policy: int, acc: np.ndarray, v: np.ndarray, loaded0=None) -> Baseline:
    """Request-level baselines of Section 5.1: 0 MaxAcc-EDF, 1 LO-EDF, 2 LO-Priority (every request alone, in order)."""
    lib, b = _load(), _Bound(w)
    n, ni = int(w.app.shape[0]), int(w.n_instances)
    per_inst = int(np.max(np.bincount(np.asarray(w.instance), minlength=ni))) if n else 0
    cap = max(1, per_inst)
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    inst = np.ascontiguousarray(w.instance, dtype=np.int32)
    arr = np.ascontiguousarray(w.arrival_ns, dtype=np.int64)
    dl = np.ascontiguousarray(w.deadline_ns, dtype=np.int64)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    t0 = np.ascontiguousarray(w.t0_ns, dtype=np.int64)
    l0 = np.full(ni, -1, dtype=np.int32) if loaded0 is None else np.ascontiguousarray(loaded0, dtype=np.int32)
    rounds = np.zeros((ni, cap), dtype=ROUND_DTYPE)
    n_rounds = np.zeros(ni, dtype=np.int64)
    reqs = np.zeros(n, dtype=REQ_DTYPE)
    t_end = np.zeros(ni, dtype=np.int64)
    l_end = np.zeros(ni, dtype=np.int32)
    margin = np.zeros(ni, dtype=np.float64)
    rc = lib.orc_baseline(C.byref(b.struct), int(policy), n, _ptr(app), _ptr(inst), _ptr(arr), _ptr(dl), _ptr(acc), _ptr(v),
                          _ptr(t0), _ptr(l0), _ptr(rounds), cap, _ptr(n_rounds), _ptr(reqs), _ptr(t_end), _ptr(l_end),
                          _ptr(margin))
    if rc != 0:
        raise ValueError("orc_baseline rejected its arguments")
    return Baseline(rounds, n_rounds, reqs, t_end, l_end, margin)


@dataclass
class WorkerDrain:
    rounds: np.ndarray      # [1, cap] ROUND_DTYPE (with the worker of every batch)
    n_rounds: np.ndarray    # [1]
    reqs: np.ndarray        # [n] REQ_DTYPE (with the worker of every request)
    t_end_ns: np.ndarray    # [W] final clock of every worker
    loaded_end: np.ndarray  # [W] model resident on every worker


def drain_workers(w, acc, v, lat_alpha_ns, lat_beta_ns, swap_ns, labels=None, loaded0: int = -1,
                  max_rounds: Optional[int] = None) -> WorkerDrain:
    """Greedy rounds on several workers (Section 6): latency arrays are [W, sumM]; one instance."""
    lib = _load()
    if int(w.n_instances) != 1:
        raise ValueError("one instance only")
    al = np.ascontiguousarray(lat_alpha_ns, dtype=np.int64)
    nw = int(al.shape[0])
    from types import SimpleNamespace
    wp = SimpleNamespace(**{**w.__dict__, "lat_alpha_ns": al, "lat_beta_ns": np.ascontiguousarray(lat_beta_ns, dtype=np.int64),
                            "swap_ns": np.ascontiguousarray(swap_ns, dtype=np.int64)})
    b = _Bound(wp)
    n = int(w.app.shape[0])
    if max_rounds is None:
        max_rounds = n + 1
    cap = max(1, min(max_rounds, n))
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    arr = np.ascontiguousarray(w.arrival_ns, dtype=np.int64)
    dl = np.ascontiguousarray(w.deadline_ns, dtype=np.int64)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    lab = None if labels is None else np.ascontiguousarray(labels, dtype=np.int32)
    rounds = np.zeros((1, cap), dtype=ROUND_DTYPE)
    n_rounds = np.zeros(1, dtype=np.int64)
    reqs = np.zeros(n, dtype=REQ_DTYPE)
    t_end = np.zeros(nw, dtype=np.int64)
    l_end = np.zeros(nw, dtype=np.int32)
    rc = lib.orc_drain_workers(C.byref(b.struct), nw, n, _ptr(app), _ptr(lab), _ptr(arr), _ptr(dl), _ptr(acc), _ptr(v),
                               int(w.t0_ns[0]), int(loaded0), int(bool(w.trace_mode)), int(max_rounds), _ptr(rounds), cap,
                               _ptr(n_rounds), _ptr(reqs), _ptr(t_end), _ptr(l_end))
    if rc != 0:
        raise ValueError("orc_drain_workers rejected its arguments")
    return WorkerDrain(rounds, n_rounds, reqs, t_end, l_end)


def score_knn(w, k: int, ref_feats: np.ndarray, ref_label: np.ndarray, ref_app: np.ndarray, want_theta: bool = False) -> Scores:
    """Scores with the k-nearest-neighbour SneakPeek model of Section 4.1 over a labelled reference set."""
    lib, b = _load(), _Bound(w)
    if int(w.n_instances) != 1:
        raise ValueError("one instance only")
    n = int(w.app.shape[0])
    mm = int(np.max(w.models_per_app))
    fdt = np.uint16 if w.feat_dtype == 1 else np.float32
    feats = np.ascontiguousarray(w.feats, dtype=fdt)
    ref = np.ascontiguousarray(ref_feats, dtype=fdt)
    rl = np.ascontiguousarray(ref_label, dtype=np.int32)
    ra = np.ascontiguousarray(ref_app, dtype=np.int32)
    app = np.ascontiguousarray(w.app, dtype=np.int32)
    acc = np.zeros((n, mm), dtype=np.float64)
    v = np.zeros(n, dtype=np.float64)
    theta = np.zeros((n, int(w.n_classes)), dtype=np.float64) if want_theta else None
    label = np.zeros(n, dtype=np.int32)
    rc = lib.orc_score_knn(C.byref(b.struct), int(k), int(ref.shape[0]), _ptr(ref), _ptr(rl), _ptr(ra), n, _ptr(feats),
                           _ptr(app), _ptr(acc), _ptr(v), _ptr(theta), _ptr(label))
    if rc != 0:
        raise ValueError("orc_score_knn rejected its arguments")
    return Scores(acc, v, theta, label)
