"""Test-only helpers: hand-built workloads and an independent replay of Eq. 1-3.

Nothing here is used by the library or by the oracle; the replay is written separately from both
so that it can serve as a pin for the schedules they emit.
"""
from __future__ import annotations

import itertools

import numpy as np

from paper_2505_06641_b200 import synth

MS = synth.MS


def manual_workload(acc_probs, recall, app, deadline_ms, alpha_ms, beta_ms, swap_ms, batch_sizes,
                    models_per_app, arrival_ms=None, t0_ms=0.0, trace_mode=False, prior_alpha=None,
                    evidence_k=0.0, tau=1.0):
    """One instance whose SneakPeek head outputs exactly the given class probabilities.

    ``acc_probs`` [n, C] are the posteriors the head must produce: the head has W = 0 on every
    feature but one, and feature 0 selects a per-request bias row, i.e. features are one-hot over
    the requests and W[a][i][c] = log p_i[c].
    """
    p = np.asarray(acc_probs, dtype=np.float64)
    n, c = p.shape
    a = len(models_per_app)
    d = max(n, 4)
    feats = np.zeros((n, d), dtype=np.float32)
    feats[np.arange(n), np.arange(n)] = 1.0
    with np.errstate(divide="ignore"):
        logp = np.maximum(np.log(p), -1.0e4)      # exp(-1e4) underflows to exactly 0
    w = np.zeros((1, a, d, c), dtype=np.float32)
    for i in range(n):
        w[0, :, i, :] = logp[i].astype(np.float32)
    ns = lambda x: np.rint(np.asarray(x, dtype=np.float64) * MS).astype(np.int64)
    arrival = ns(np.zeros(n) if arrival_ms is None else arrival_ms)
    return synth.Workload(
        name="manual", n_instances=1, n_apps=a, n_classes=c, feat_dim=d, feat_dtype=synth.F32,
        models_per_app=np.asarray(models_per_app, dtype=np.int32), head_w=w,
        head_b=np.zeros((1, a, c), dtype=np.float32), recall=np.asarray(recall, dtype=np.float32)[None],
        lat_alpha_ns=ns(alpha_ms)[None], lat_beta_ns=ns(beta_ms)[None], swap_ns=ns(swap_ms)[None],
        batch_sizes=np.asarray(batch_sizes, dtype=np.int32),
        penalty_kind=np.zeros(a, dtype=np.int32), prio_time_scale_s=tau, feats=feats,
        app=np.asarray(app, dtype=np.int32), arrival_ns=arrival, deadline_ns=ns(deadline_ms),
        instance=np.zeros(n, dtype=np.int32), t0_ns=ns([t0_ms]), trace_mode=trace_mode,
        prior_alpha=None if prior_alpha is None else np.asarray(prior_alpha, dtype=np.float32)[None],
        evidence_k=evidence_k)


def one_instance(w, k):
    """Instance ``k`` of a batched workload as a workload of its own."""
    sel = np.nonzero(np.asarray(w.instance) == k)[0]
    return synth.Workload(
        name=w.name, n_instances=1, n_apps=w.n_apps, n_classes=w.n_classes, feat_dim=w.feat_dim,
        feat_dtype=w.feat_dtype, models_per_app=w.models_per_app, head_w=w.head_w[k:k + 1],
        head_b=w.head_b[k:k + 1], recall=w.recall[k:k + 1], lat_alpha_ns=w.lat_alpha_ns[k:k + 1],
        lat_beta_ns=w.lat_beta_ns[k:k + 1], swap_ns=w.swap_ns[k:k + 1], batch_sizes=w.batch_sizes,
        penalty_kind=w.penalty_kind, prio_time_scale_s=w.prio_time_scale_s, feats=w.feats[sel],
        app=w.app[sel], arrival_ns=w.arrival_ns[sel], deadline_ns=w.deadline_ns[sel],
        instance=np.zeros(len(sel), dtype=np.int32), t0_ns=w.t0_ns[k:k + 1], trace_mode=w.trace_mode,
        prior_alpha=None if w.prior_alpha is None else w.prior_alpha[k:k + 1], evidence_k=w.evidence_k)


def first_model(w, a):
    return int(np.sum(w.models_per_app[:a]))


def replay_schedule(w, acc, reqs, rounds, n_rounds, loaded0=-1, inst=0):
    """Independent check of an emitted schedule of one instance against Eq. 1-3.

    Walks the requests in their emitted execution order s_ij, rebuilds every batch's completion
    time from the latency profile alone (start time = sum of the latencies of everything ordered
    ahead, Eq. 1, with the swap time charged whenever the model changes), applies the step
    penalty to each member (Eq. 2) and returns the total utility (the sum inside Eq. 3).
    Raises AssertionError when the records are inconsistent with that replay.
    """
    sel = np.nonzero(np.asarray(w.instance) == inst)[0]
    sm = w.sum_models
    al, be, sw = w.lat_alpha_ns[inst], w.lat_beta_ns[inst], w.swap_ns[inst]
    sched = [i for i in sel if reqs["status"][i] == 1]
    sched.sort(key=lambda i: reqs["order"][i])
    orders = [int(reqs["order"][i]) for i in sched]
    assert orders == list(range(1, len(sched) + 1)), "execution orders must be 1..K without gaps"
    total, prev_model, clock, pos = 0.0, loaded0, int(w.t0_ns[inst]), 0
    for r in range(int(n_rounds)):
        rec = rounds[r]
        members = []
        while pos < len(sched) and reqs["round"][sched[pos]] == r:
            members.append(sched[pos]); pos += 1
        assert len(members) == rec["n_members"] >= 1
        g = int(rec["model"])
        a = int(rec["app"])
        assert 0 <= g < sm and first_model(w, a) <= g < first_model(w, a) + w.models_per_app[a]
        assert all(reqs["model"][i] == g and w.app[i] == a for i in members)
        keys = [(int(w.deadline_ns[i]), int(i)) for i in members]
        assert keys == sorted(keys), "members run in (deadline, id) order"
        start = int(rec["t_start_ns"])
        if w.trace_mode:
            assert start >= clock
            if start > clock:          # an idle scheduler may only wake at an arrival
                assert start in set(int(x) for x in w.arrival_ns[sel])
        else:
            assert start == clock
        end = start + (int(sw[g]) if g != prev_model else 0) + int(al[g]) + int(be[g]) * len(members)
        assert end == rec["t_end_ns"]
        j = g - first_model(w, a)
        kind = int(w.penalty_kind[a])
        if kind == 0:
            u = sum(float(acc[i, j]) for i in members if not (w.deadline_ns[i] < end))
        else:                              # utility degrades over the relative deadline after the deadline (Section 5.1)
            u = 0.0
            for i in members:
                d, delta = int(w.deadline_ns[i]), int(w.deadline_ns[i]) - int(w.arrival_ns[i])
                late = min(max((end - d) / delta, 0.0), 1.0) if delta > 0 else float(d < end)
                gamma = late if kind == 1 else (0.0 if late <= 0 else 1.0 if late >= 1 else 1.0 / (1.0 + ((1.0 - late) / late) ** 3))
                u += float(acc[i, j]) * (1.0 - gamma)
        assert abs(u - rec["utility"]) <= 1e-11 * max(1.0, abs(u))
        total += u
        clock, prev_model = end, g
    assert pos == len(sched)
    return total


def brute_force_request_level(w, acc, loaded0=-1):
    """Exhaustive optimum of Eq. 3-6 for one application-agnostic tiny queue with batch size 1.

    Enumerates every execution order and every model assignment (n! * prod |M_a_i| solutions),
    evaluates each by Eq. 1-2 with the step penalty, and returns (best total utility, number of
    solutions visited).
    """
    n = w.n_requests
    al, be, sw = w.lat_alpha_ns[0], w.lat_beta_ns[0], w.swap_ns[0]
    best, count = -1.0, 0
    choices = [range(first_model(w, int(a)), first_model(w, int(a)) + int(w.models_per_app[a])) for a in w.app]
    for perm in itertools.permutations(range(n)):
        for models in itertools.product(*[choices[i] for i in perm]):
            count += 1
            t, prev, tot = int(w.t0_ns[0]), loaded0, 0.0
            for i, g in zip(perm, models):
                t += (int(sw[g]) if g != prev else 0) + int(al[g]) + int(be[g])
                prev = g
                if not (w.deadline_ns[i] < t):
                    tot += float(acc[i, g - first_model(w, int(w.app[i]))])
            best = max(best, tot)
    return best, count
