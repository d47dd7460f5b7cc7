"""Seeded synthetic workloads for the SneakPeek scoring-and-selection path.

This module only DRAWS inputs (features, heads, profiles, arrivals, deadlines).  It holds none of
the method's arithmetic: no softmax, no accuracy contraction, no priority, no utility, no
scheduling.  Both the CPU oracle's tests and the CUDA library's tests/benchmark take their inputs
from here so that the two sides see identical bytes.

The five workloads keep the structure of the paper's evaluation set-up (Section 5.1: three
applications, a handful of model variants per application that trade latency for accuracy,
per-label accuracy profiles, deadlines a few hundred ms after arrival, requests spread over a
scheduling window) but every value is synthetic; nothing of the paper's datasets is reproduced.

All times are int64 nanoseconds (millisecond draws are rounded to the nearest ns).
``N(0, s)`` means standard deviation ``s``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

MS = 1_000_000  # ns per ms

F32 = 0
BF16 = 1

PEN_STEP = 0
PEN_LINEAR = 1
PEN_SIGMOID = 2


@dataclass
class Workload:
    """Inputs of one scoring + scheduling job (possibly many independent instances).

    Profile arrays carry a leading instance axis ``I`` (``I == 1`` for a single scheduler).
    Request arrays are flat over all instances, grouped by instance in ascending order, and
    inside an instance ordered by arrival time.
    """

    name: str
    n_instances: int
    n_apps: int
    n_classes: int
    feat_dim: int
    feat_dtype: int                 # F32 or BF16 (bf16 stored as uint16 bit patterns)
    models_per_app: np.ndarray      # [A] int32
    head_w: np.ndarray              # [I, A, D, C] float32, or uint16 (bf16 bits) when feat_dtype == BF16
    head_b: np.ndarray              # [I, A, C] float32
    recall: np.ndarray              # [I, sumM, C] float32 per-model per-class accuracy
    lat_alpha_ns: np.ndarray        # [I, sumM] int64
    lat_beta_ns: np.ndarray         # [I, sumM] int64
    swap_ns: np.ndarray             # [I, sumM] int64
    batch_sizes: np.ndarray         # [nB] int32 ascending
    penalty_kind: np.ndarray        # [A] int32
    prio_time_scale_s: float
    feats: np.ndarray               # [N, D] float32 or uint16 (bf16 bits)
    app: np.ndarray                 # [N] int32
    arrival_ns: np.ndarray          # [N] int64
    deadline_ns: np.ndarray         # [N] int64
    instance: np.ndarray            # [N] int32
    t0_ns: np.ndarray               # [I] int64 initial clock
    trace_mode: bool                # False: every request is pending at t0; True: requests join at arrival <= clock
    prior_alpha: Optional[np.ndarray] = None   # [I, A, C] float32 or None
    evidence_k: float = 0.0
    meta: Dict[str, object] = field(default_factory=dict)

    @property
    def n_requests(self) -> int:
        return int(self.app.shape[0])

    @property
    def sum_models(self) -> int:
        return int(self.models_per_app.sum())

    @property
    def max_models(self) -> int:
        return int(self.models_per_app.max())


# ----------------------------------------------------------------------------------------------
# bf16 helpers (storage format only: round-to-nearest-even truncation of the fp32 bit pattern)
# ----------------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns to float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _ms_to_ns(x) -> np.ndarray:
    return np.rint(np.asarray(x, dtype=np.float64) * MS).astype(np.int64)


def _pow2_batches(bmax: int) -> np.ndarray:
    out, b = [], 1
    while b <= bmax:
        out.append(b)
        b *= 2
    return np.asarray(out, dtype=np.int32)


# ----------------------------------------------------------------------------------------------
# per-instance draws
# ----------------------------------------------------------------------------------------------

@dataclass
class _Spec:
    n_apps: int
    models: int
    n_classes: int
    n_requests: int
    feat_dim: int
    feat_dtype: int
    w_std: float
    recall: str                 # "uniform", "beta82", "beta52_hard"
    alpha_ms: tuple
    beta_ms: tuple
    swap_ms: tuple
    bmax: int
    arrivals: str               # "poisson200", "window20", "window10", "bursty"
    deadline_ms: tuple
    infeasible_frac: float = 0.0
    zipf_features: bool = False
    trace_mode: bool = False


def _draw_recall(rng: np.random.Generator, spec: _Spec, sum_m: int) -> np.ndarray:
    a, m, c = spec.n_apps, spec.models, spec.n_classes
    if spec.recall == "uniform":
        return rng.uniform(0.5, 0.99, size=(sum_m, c)).astype(np.float32)
    if spec.recall == "beta82":
        return rng.beta(8.0, 2.0, size=(sum_m, c)).astype(np.float32)
    if spec.recall == "beta52_hard":
        r = rng.beta(5.0, 2.0, size=(sum_m, c))
        n_hard = max(1, int(round(0.05 * c)))
        for app in range(a):                       # the same hard classes for every model of an app
            hard = rng.choice(c, size=n_hard, replace=False)
            r[app * m:(app + 1) * m, hard] = rng.uniform(0.05, 0.15, size=(m, n_hard))
        return r.astype(np.float32)
    raise ValueError(spec.recall)


def _draw_arrivals_ms(rng: np.random.Generator, spec: _Spec, n: int) -> np.ndarray:
    if spec.arrivals == "poisson200":              # Poisson process, 200 req/s
        return np.cumsum(rng.exponential(5.0, size=n))
    if spec.arrivals == "window20":
        return np.sort(rng.uniform(0.0, 20.0, size=n))
    if spec.arrivals == "window10":
        return np.sort(rng.uniform(0.0, 10.0, size=n))
    if spec.arrivals == "bursty":                  # rate alternates 100 / 5000 req/s every 2 s
        lam = np.cumsum(rng.exponential(1.0, size=n))          # unit-rate process = cumulative intensity
        per_period = 100.0 * 2.0 + 5000.0 * 2.0
        period = np.floor(lam / per_period)
        rem = lam - period * per_period
        t_s = np.where(rem < 200.0, period * 4.0 + rem / 100.0,
                       period * 4.0 + 2.0 + (rem - 200.0) / 5000.0)
        return t_s * 1000.0
    raise ValueError(spec.arrivals)


def _draw_features(rng: np.random.Generator, spec: _Spec, n: int) -> np.ndarray:
    d = spec.feat_dim
    if not spec.zipf_features:
        x = rng.standard_normal(size=(n, d), dtype=np.float32)
    else:
        c = spec.n_classes
        pk = (np.arange(1, c + 1, dtype=np.float64)) ** -1.1      # Zipf(1.1) truncated to C labels
        pk /= pk.sum()
        label = rng.choice(c, size=n, p=pk)
        mu = (0.25 * rng.standard_normal(size=(c, d), dtype=np.float32)).astype(np.float32)
        x = np.empty((n, d), dtype=np.float32)
        step = 8192
        for s in range(0, n, step):
            e = min(n, s + step)
            x[s:e] = mu[label[s:e]] + rng.standard_normal(size=(e - s, d), dtype=np.float32)
    if spec.feat_dtype == BF16:
        return f32_to_bf16_bits(x)
    return x


def _draw_instance(seed: int, spec: _Spec):
    """All draws of one instance, in a fixed order, from its own generator."""
    rng = np.random.default_rng(seed)
    a, m, c, d, n = spec.n_apps, spec.models, spec.n_classes, spec.feat_dim, spec.n_requests
    sum_m = a * m
    w = (spec.w_std * rng.standard_normal(size=(a, d, c), dtype=np.float32)).astype(np.float32)
    b = (spec.w_std * rng.standard_normal(size=(a, c), dtype=np.float32)).astype(np.float32)
    if spec.feat_dtype == BF16:
        w = f32_to_bf16_bits(w)
    recall = _draw_recall(rng, spec, sum_m)
    alpha = _ms_to_ns(rng.uniform(*spec.alpha_ms, size=sum_m))
    beta = _ms_to_ns(rng.uniform(*spec.beta_ms, size=sum_m))
    swap = _ms_to_ns(rng.uniform(*spec.swap_ms, size=sum_m))
    app = rng.integers(0, a, size=n, dtype=np.int32)
    arr_ms = _draw_arrivals_ms(rng, spec, n)
    arrival = _ms_to_ns(arr_ms)
    deadline = arrival + _ms_to_ns(rng.uniform(*spec.deadline_ms, size=n))
    t0 = int(arrival[0]) if spec.trace_mode else int(arrival.max())
    if spec.infeasible_frac > 0.0:
        k = int(round(spec.infeasible_frac * n))
        idx = rng.choice(n, size=k, replace=False)
        deadline[idx] = t0 - _ms_to_ns(rng.uniform(0.0, 100.0, size=k))
    feats = _draw_features(rng, spec, n)
    return dict(w=w, b=b, recall=recall, alpha=alpha, beta=beta, swap=swap, app=app,
                arrival=arrival, deadline=deadline, t0=t0, feats=feats)


_SPECS = {
    # name: (spec, base seed, instances)
    "C1": (_Spec(3, 4, 10, 256, 64, F32, 0.1, "uniform", (2, 20), (0.5, 5), (50, 500), 32,
                 "poisson200", (50, 500)), 0, 1),
    "C2": (_Spec(3, 8, 100, 4096, 256, F32, 0.05, "beta82", (1, 30), (0.2, 8), (20, 800), 64,
                 "window20", (20, 1000), infeasible_frac=0.30), 1, 1),
    "C3": (_Spec(3, 16, 1000, 65536, 1024, BF16, 0.03, "beta52_hard", (1, 30), (0.2, 8), (20, 800), 128,
                 "window10", (10, 2000), zipf_features=True), 2, 1),
    "C4": (_Spec(3, 6, 20, 512, 128, F32, 0.1, "uniform", (2, 20), (0.5, 5), (50, 500), 32,
                 "poisson200", (50, 500)), 1000, 16384),
    "C5": (_Spec(3, 12, 200, 1_000_000, 512, F32, 0.05, "beta82", (1, 30), (0.2, 8), (20, 800), 64,
                 "bursty", (20, 800), trace_mode=True), 3, 1),
}

CONFIG_NAMES = tuple(_SPECS)


def make_workload(name: str, n_requests: Optional[int] = None, n_instances: Optional[int] = None,
                  first_instance: int = 0, **overrides) -> Workload:
    """Draw one of the five workloads ("C1".."C5").

    ``n_requests`` (per instance) and ``n_instances`` shrink or grow a workload without changing
    its recipe; instance ``i`` always uses seed ``base_seed + first_instance + i`` so a subset of
    the batched workload equals the same instances of the full one.  ``overrides`` replace fields
    of the recipe (for test variants, e.g. ``models=2``).
    """
    spec0, base_seed, inst0 = _SPECS[name]
    spec = _Spec(**{**spec0.__dict__, **overrides})
    if n_requests is not None:
        spec.n_requests = int(n_requests)
    n_inst = int(n_instances) if n_instances is not None else inst0
    parts = [_draw_instance(base_seed + first_instance + i, spec) for i in range(n_inst)]
    a, m = spec.n_apps, spec.models
    n = spec.n_requests
    stack = lambda k: np.stack([p[k] for p in parts])
    cat = lambda k: np.concatenate([p[k] for p in parts])
    return Workload(
        name=name, n_instances=n_inst, n_apps=a, n_classes=spec.n_classes, feat_dim=spec.feat_dim,
        feat_dtype=spec.feat_dtype, models_per_app=np.full(a, m, dtype=np.int32),
        head_w=stack("w"), head_b=stack("b"), recall=stack("recall"),
        lat_alpha_ns=stack("alpha"), lat_beta_ns=stack("beta"), swap_ns=stack("swap"),
        batch_sizes=_pow2_batches(spec.bmax), penalty_kind=np.full(a, PEN_STEP, dtype=np.int32),
        prio_time_scale_s=1.0, feats=cat("feats"), app=cat("app"), arrival_ns=cat("arrival"),
        deadline_ns=cat("deadline"),
        instance=np.repeat(np.arange(n_inst, dtype=np.int32), n),
        t0_ns=np.asarray([p["t0"] for p in parts], dtype=np.int64), trace_mode=spec.trace_mode,
        meta=dict(base_seed=base_seed, first_instance=first_instance, requests_per_instance=n),
    )


def with_short_circuit(w: Workload, static_acc) -> Workload:
    """Adds the short-circuit candidate of the paper's Section 4.3 to every application of ``w``.

    The candidate is one more model variant per application, placed after the application's own variants: it
    answers at once (latency alpha = beta = 0, no swap time) and its accuracy is the profiled, static accuracy
    ``static_acc[a]`` whatever the request looks like.  In the profile format that is a recall row that holds the
    same value for every label.  Only profile arrays change; requests, heads and seeds stay as they are.
    """
    a, ni = int(w.n_apps), int(w.n_instances)
    acc = np.broadcast_to(np.asarray(static_acc, dtype=np.float32), (a,))
    old_m = np.asarray(w.models_per_app, dtype=np.int64)
    first = np.concatenate([[0], np.cumsum(old_m)])
    c = int(w.n_classes)

    def grow(arr, fill_rows):
        out = []
        for app in range(a):
            out.append(arr[:, first[app]:first[app + 1]])
            out.append(fill_rows[app])
        return np.ascontiguousarray(np.concatenate(out, axis=1))

    recall = grow(w.recall, [np.full((ni, 1, c), acc[app], dtype=np.float32) for app in range(a)])
    zeros = [np.zeros((ni, 1), dtype=np.int64) for _ in range(a)]
    out = Workload(**{**w.__dict__})
    out.models_per_app = (old_m + 1).astype(np.int32)
    out.recall = recall
    out.lat_alpha_ns = grow(w.lat_alpha_ns, zeros)
    out.lat_beta_ns = grow(w.lat_beta_ns, zeros)
    out.swap_ns = grow(w.swap_ns, zeros)
    out.meta = dict(w.meta, short_circuit=[float(x) for x in acc])
    return out
