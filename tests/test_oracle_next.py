"""Pins of the oracle's data-aware sub-groups (Section 4.3), of Algorithm 1's exhaustive branch and of the request-level
baselines of Section 5.1: the cases of the paper's group-splitting figure, hand-worked totals, the solution count of
Section 3.1, an independent Python enumerator and the independent replay of Eq. 1-3."""
import math

import numpy as np
import pytest

from oracle import oracle
from helpers import MS, brute_force_request_level, first_model, manual_workload, replay_schedule


def _split_run(w):
    s = oracle.score(w)
    return s, oracle.drain(w, s.acc, s.v), oracle.drain(w, s.acc, s.v, labels=s.label)


def _two_task_workload(probs_a, probs_b, **kw):
    """Two binary tasks (applications) with two models each: model 0 of a task is good on label 0, model 1 on label 1."""
    probs = list(probs_a) + list(probs_b)
    n = len(probs)
    args = dict(recall=[[0.9, 0.2], [0.3, 0.95], [0.85, 0.1], [0.15, 0.8]], app=[0] * len(probs_a) + [1] * len(probs_b),
                deadline_ms=[5000 + 10 * i for i in range(n)], alpha_ms=[5, 6, 7, 8], beta_ms=[1, 1, 1, 1],
                swap_ms=[0, 0, 0, 0], batch_sizes=[1, 2, 4, 8], models_per_app=[2, 2])
    args.update(kw)
    return manual_workload(probs, **args)


def test_labels_follow_the_half_threshold():
    w = manual_workload([[0.9, 0.1], [0.2, 0.8], [0.5, 0.5], [0.4, 0.35, 0.25][:2] + [0.0]][:3] + [[0.5, 0.5]],
                        [[0.8, 0.8]], app=[0] * 4, deadline_ms=[1000] * 4, alpha_ms=[1], beta_ms=[1], swap_ms=[0],
                        batch_sizes=[1], models_per_app=[1])
    s = oracle.score(w)
    assert list(s.label) == [0, 1, -1, -1]                        # exactly one half is not "more than a half"
    w3 = manual_workload([[0.4, 0.35, 0.25], [0.1, 0.3, 0.6]], [[0.8, 0.8, 0.8]], app=[0, 0], deadline_ms=[1000] * 2,
                         alpha_ms=[1], beta_ms=[1], swap_ms=[0], batch_sizes=[1], models_per_app=[1])
    assert list(oracle.score(w3).label) == [-1, 2]                # multi-class: inconclusive stays unsplit


def test_figure_case_same_class_is_not_split_and_two_classes_are():
    """The two cases of the group-splitting figure: a task whose requests all indicate one class stays one group; a task
    whose requests indicate both classes becomes two sub-groups, each served on the model that suits its class."""
    w = _two_task_workload([[0.9, 0.1], [0.8, 0.2], [0.95, 0.05]], [[0.9, 0.1], [0.15, 0.85], [0.8, 0.2], [0.1, 0.9]])
    s, plain, split = _split_run(w)
    assert list(s.label) == [0, 0, 0, 0, 1, 0, 1]
    r = split.rounds[0, :int(split.n_rounds[0])]
    task_a, task_b = r[r["app"] == 0], r[r["app"] == 1]
    assert len(task_a) == 1 and task_a["n_members"][0] == 3 and task_a["label"][0] == 0
    assert sorted(task_b["label"]) == [0, 1] and sorted(task_b["n_members"]) == [2, 2]
    for rec in task_b:                                          # members of a round share the label; the model fits it
        members = [i for i in range(w.n_requests) if split.reqs["round"][i] == rec["round"]]
        assert all(s.label[i] == rec["label"] for i in members)
        assert rec["model"] == first_model(w, 1) + rec["label"]
    # without splitting, task b runs as one batch on one model
    rp = plain.rounds[0, :int(plain.n_rounds[0])]
    assert len(rp[rp["app"] == 1]) == 1 and np.all(rp["label"] == -1)
    assert split.rounds["utility"].sum() > plain.rounds["utility"].sum()


def test_split_total_of_a_hand_worked_case():
    """One task, one-hot posteriors, model 0 right on label 0 only and model 1 on label 1 only: unsplit, the batch of
    both requests earns 0.9 + 0.1 on either model; split, each request runs on its own model and earns 0.9."""
    w = manual_workload([[1.0, 0.0], [0.0, 1.0]], [[0.9, 0.1], [0.1, 0.9]], app=[0, 0], deadline_ms=[1000, 1001],
                        alpha_ms=[1, 1], beta_ms=[1, 1], swap_ms=[0, 0], batch_sizes=[1, 2], models_per_app=[2])
    s, plain, split = _split_run(w)
    assert plain.rounds["utility"].sum() == pytest.approx(1.0, abs=1e-6)            # recall is stored as float
    assert split.rounds["utility"].sum() == pytest.approx(1.8, abs=1e-6)
    assert [int(x) for x in split.reqs["model"]] == [0, 1]


@pytest.mark.parametrize("seed", range(4))
def test_no_split_when_labels_are_inconclusive_or_uniform_per_task(seed):
    """Sub-groups reduce to the applications when no posterior passes one half, and when every request of a task
    indicates the same class: the schedule is then the unsplit one, round by round."""
    rng = np.random.default_rng(300 + seed)
    n, c = 40, 5
    flat = rng.dirichlet(np.ones(c) * 8.0, size=n)               # no entry above one half
    assert flat.max() < 0.5
    app = rng.integers(0, 3, size=n)
    peaked = np.full((n, c), 0.05)
    peaked[np.arange(n), app] = 0.8                              # task a always indicates class a
    for probs in (flat, peaked):
        w = manual_workload(probs, rng.uniform(0.3, 0.99, size=(6, c)), app=app, deadline_ms=rng.uniform(50, 900, size=n),
                            alpha_ms=rng.uniform(2, 20, size=6), beta_ms=rng.uniform(0.5, 5, size=6),
                            swap_ms=rng.uniform(5, 50, size=6), batch_sizes=[1, 2, 4, 8], models_per_app=[2, 2, 2])
        s, plain, split = _split_run(w)
        assert plain.n_rounds[0] == split.n_rounds[0] and np.array_equal(plain.reqs, split.reqs)
        k = int(plain.n_rounds[0])
        for f in ("app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns", "utility", "group_priority"):
            assert np.array_equal(plain.rounds[0, :k][f], split.rounds[0, :k][f]), f


def test_split_schedule_replays_under_eq_1_to_3():
    rng = np.random.default_rng(7)
    n, c = 60, 4
    probs = rng.dirichlet(np.ones(c) * 0.3, size=n)              # mostly confident posteriors
    w = manual_workload(probs, rng.uniform(0.2, 0.99, size=(6, c)), app=rng.integers(0, 2, size=n),
                        deadline_ms=rng.uniform(30, 600, size=n), alpha_ms=rng.uniform(2, 20, size=6),
                        beta_ms=rng.uniform(0.5, 5, size=6), swap_ms=rng.uniform(5, 50, size=6), batch_sizes=[1, 2, 4, 8],
                        models_per_app=[3, 3])
    s, plain, split = _split_run(w)
    assert len(set(s.label)) > 2
    k = int(split.n_rounds[0])
    total = replay_schedule(w, s.acc, split.reqs, split.rounds[0], k)
    assert total == pytest.approx(split.rounds[0, :k]["utility"].sum(), rel=1e-12)
    for rec in split.rounds[0, :k]:                              # a round never mixes sub-groups
        members = [i for i in range(n) if split.reqs["round"][i] == rec["round"] and split.reqs["status"][i] == 1]
        assert len({(int(w.app[i]), int(s.label[i])) for i in members}) == 1


# ------------------------------------------------------------------ exhaustive branch of Algorithm 1

def _bf_workload(rng, n, a, m, bmax=4, c=3, deadline=(30, 400)):
    return manual_workload(rng.dirichlet(np.ones(c), size=n), rng.uniform(0.2, 0.99, size=(a * m, c)),
                           app=np.concatenate([np.arange(a), rng.integers(0, a, size=n - a)]),
                           deadline_ms=rng.uniform(*deadline, size=n), alpha_ms=rng.uniform(2, 20, size=a * m),
                           beta_ms=rng.uniform(0.5, 5, size=a * m), swap_ms=rng.uniform(5, 80, size=a * m),
                           batch_sizes=[1, 2, bmax], models_per_app=[m] * a)


def _eval_group_solution(w, acc, order, models):
    """Total utility of serving the applications in `order` with models[a], whole, in batches of the largest size."""
    t, loaded, total, bmax = int(w.t0_ns[0]), -1, 0.0, int(w.batch_sizes[-1])
    for a in order:
        members = sorted([i for i in range(w.n_requests) if w.app[i] == a], key=lambda i: (int(w.deadline_ns[i]), i))
        g = first_model(w, a) + models[a]
        for k0 in range(0, len(members), bmax):
            batch = members[k0:k0 + bmax]
            t += (int(w.swap_ns[0, g]) if g != loaded else 0) + int(w.lat_alpha_ns[0, g]) + int(w.lat_beta_ns[0, g]) * len(batch)
            loaded = g
            total += sum(float(acc[i, models[a]]) for i in batch if not (w.deadline_ns[i] < t))
    return total


@pytest.mark.parametrize("seed", range(5))
def test_exhaustive_branch_finds_the_best_group_level_solution(seed):
    import itertools
    rng = np.random.default_rng(500 + seed)
    a, m = int(rng.integers(2, 4)), int(rng.integers(2, 4))
    w = _bf_workload(rng, 14, a, m)
    s = oracle.score(w)
    bf = oracle.bruteforce(w, s.acc)
    assert bf.n_solutions == math.factorial(a) * m ** a
    best = max(_eval_group_solution(w, s.acc, order, models)
               for order in itertools.permutations(range(a)) for models in itertools.product(range(m), repeat=a))
    assert bf.total == pytest.approx(best, rel=1e-12)
    k = int(bf.n_rounds[0])
    assert bf.rounds[0, :k]["utility"].sum() == pytest.approx(best, rel=1e-12)
    assert np.all(bf.reqs["status"] == oracle.SCHEDULED)
    assert replay_schedule(w, s.acc, bf.reqs, bf.rounds[0], k) == pytest.approx(best, rel=1e-12)
    # the greedy branch serves the same groups one batch at a time; whenever it neither retires a request nor
    # interleaves the groups, its schedule is one of the solutions enumerated, so it cannot do better
    g = oracle.drain(w, s.acc, s.v)
    apps = [int(x) for x in g.rounds[0, :int(g.n_rounds[0])]["app"]]
    contiguous = all(apps[i] == apps[i - 1] or apps[i] not in apps[:i] for i in range(1, len(apps)))
    full = all(int(r["n_members"]) == int(w.batch_sizes[-1]) or i + 1 == len(apps) or apps[i + 1] != apps[i]
               for i, r in enumerate(g.rounds[0, :len(apps)]))
    if np.all(g.reqs["status"] == oracle.SCHEDULED) and contiguous and full:
        assert g.rounds[0, :len(apps)]["utility"].sum() <= bf.total * (1 + 1e-12)


def test_exhaustive_branch_equals_the_request_level_optimum_for_singleton_groups():
    """One request per application and batch size 1: the group-level problem is the request-level problem of
    Section 3.1, whose n! |M|^n solutions an independent enumerator visits."""
    rng = np.random.default_rng(11)
    n, m = 4, 2
    w = manual_workload(rng.dirichlet(np.ones(3), size=n), rng.uniform(0.2, 0.99, size=(n * m, 3)), app=np.arange(n),
                        deadline_ms=rng.uniform(20, 120, size=n), alpha_ms=rng.uniform(5, 30, size=n * m),
                        beta_ms=rng.uniform(1, 10, size=n * m), swap_ms=rng.uniform(5, 40, size=n * m), batch_sizes=[1],
                        models_per_app=[m] * n)
    s = oracle.score(w)
    bf = oracle.bruteforce(w, s.acc)
    best, count = brute_force_request_level(w, s.acc)
    assert count == math.factorial(n) * m ** n == bf.n_solutions
    assert bf.total == pytest.approx(best, rel=1e-12)


def test_exhaustive_branch_ties_go_to_the_first_solution():
    """Two identical models: the lower one is chosen; two identical groups: the lower application goes first."""
    w = manual_workload([[0.5, 0.5]] * 4, [[0.8, 0.8]] * 4, app=[0, 1, 0, 1], deadline_ms=[1e6] * 4, alpha_ms=[5] * 4,
                        beta_ms=[1] * 4, swap_ms=[0] * 4, batch_sizes=[4], models_per_app=[2, 2])
    s = oracle.score(w)
    bf = oracle.bruteforce(w, s.acc)
    assert [int(x) for x in bf.rounds[0, :2]["app"]] == [0, 1] and [int(x) for x in bf.rounds[0, :2]["model"]] == [0, 2]
    assert bf.second == -np.inf and bf.n_solutions == 8


def test_exhaustive_branch_over_sub_groups_and_its_limits():
    w = _two_task_workload([[0.9, 0.1], [0.2, 0.8]], [[0.9, 0.1], [0.15, 0.85], [0.45, 0.55]])
    s = oracle.score(w)
    bf = oracle.bruteforce(w, s.acc, labels=s.label)
    assert bf.n_solutions == math.factorial(4) * 2 ** 4
    assert sorted(zip(bf.rounds[0, :4]["app"], bf.rounds[0, :4]["label"])) == [(0, 0), (0, 1), (1, 0), (1, 1)]
    assert bf.total >= oracle.bruteforce(w, s.acc).total - 1e-12
    rng = np.random.default_rng(3)
    big = manual_workload(rng.dirichlet(np.ones(2), size=9), rng.uniform(0.2, 0.9, size=(9, 2)), app=np.arange(9),
                          deadline_ms=[100] * 9, alpha_ms=[1] * 9, beta_ms=[1] * 9, swap_ms=[0] * 9, batch_sizes=[1],
                          models_per_app=[1] * 9)
    with pytest.raises(ValueError):
        oracle.bruteforce(big, oracle.score(big).acc)


# ------------------------------------------------------------------ request-level baselines

def _baseline_workload(rng, n=30, kinds=None, deadline=(20, 300)):
    a, m, c = 3, 3, 4
    w = manual_workload(rng.dirichlet(np.ones(c), size=n), rng.uniform(0.2, 0.99, size=(a * m, c)),
                        app=rng.integers(0, a, size=n), deadline_ms=rng.uniform(*deadline, size=n),
                        alpha_ms=rng.uniform(2, 20, size=a * m), beta_ms=rng.uniform(0.5, 5, size=a * m),
                        swap_ms=rng.uniform(5, 50, size=a * m), batch_sizes=[1, 2], models_per_app=[m] * a)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    return w


@pytest.mark.parametrize("policy", [oracle.MAXACC_EDF, oracle.LO_EDF, oracle.LO_PRIORITY])
@pytest.mark.parametrize("kinds", [None, [1, 2, 0]])
def test_baseline_schedules_replay_and_follow_their_order(policy, kinds):
    rng = np.random.default_rng(40 + policy)
    w = _baseline_workload(rng, kinds=kinds)
    s = oracle.score(w)
    b = oracle.baseline(w, policy, s.acc, s.v)
    n = w.n_requests
    assert b.n_rounds[0] == n and np.all(b.reqs["status"] == oracle.SCHEDULED)
    total = replay_schedule(w, s.acc, b.reqs, b.rounds[0], n)    # Eq. 1-3 over the emitted s_ij
    assert total == pytest.approx(b.rounds[0]["utility"].sum(), rel=1e-12)
    by_order = np.argsort(b.reqs["order"])
    if policy == oracle.LO_PRIORITY:
        prio = s.v * np.exp(-(w.deadline_ns - w.t0_ns[0]) * 1e-9 / w.prio_time_scale_s)
        assert np.all(np.diff(prio[by_order]) <= 0)
    else:
        keys = [(int(w.deadline_ns[i]), int(i)) for i in by_order]
        assert keys == sorted(keys)
    # every request got the model its policy asks for at the moment it started
    loaded = -1
    for pos, i in enumerate(by_order):
        rec = b.rounds[0, pos]
        a = int(w.app[i]); g0 = first_model(w, a)
        ends = [int(rec["t_start_ns"]) + (int(w.swap_ns[0, g0 + j]) if g0 + j != loaded else 0) + int(w.lat_alpha_ns[0, g0 + j])
                + int(w.lat_beta_ns[0, g0 + j]) for j in range(3)]
        if policy == oracle.MAXACC_EDF:
            ok = [j for j in range(3) if not (w.deadline_ns[i] < ends[j])] or list(range(3))
            want = max(ok, key=lambda j: (s.acc[i, j], -j))
        else:
            kind = int(w.penalty_kind[a])
            util = [s.acc[i, j] * (1.0 - oracle.penalty(kind, int(w.deadline_ns[i]), int(w.arrival_ns[i]), ends[j])) for j in range(3)]
            want = max(range(3), key=lambda j: (util[j], -j))
        assert int(rec["model"]) == g0 + want
        loaded = int(rec["model"])


def test_baselines_on_a_hand_worked_queue():
    """Two models: 0 is fast and poor (10 ms, 0.6), 1 slow and good (50 ms, 0.9).  Request 0 (deadline 30 ms) can only
    be met by model 0; request 1 (deadline 200 ms) by both; request 2 (deadline 20 ms) by none once request 0 ran."""
    w = manual_workload([[1.0, 0.0]] * 3, [[0.6, 0.6], [0.9, 0.9]], app=[0, 0, 0], deadline_ms=[30, 200, 20],
                        alpha_ms=[5, 45], beta_ms=[5, 5], swap_ms=[0, 0], batch_sizes=[1], models_per_app=[2])
    s = oracle.score(w)
    for policy in (oracle.MAXACC_EDF, oracle.LO_EDF):
        b = oracle.baseline(w, policy, s.acc, s.v)
        # EDF: request 2 (20 ms) first, met by model 0 at 10 ms; request 0 (30 ms) met by model 0 at 20 ms;
        # request 1 (200 ms) takes the good model, done at 70 ms
        assert [int(x) for x in np.argsort(b.reqs["order"])] == [2, 0, 1]
        assert [int(b.reqs["model"][i]) for i in (2, 0, 1)] == [0, 0, 1]
        assert b.rounds[0]["utility"].sum() == pytest.approx(0.6 + 0.6 + 0.9, abs=1e-6)
    w.deadline_ns[2] = 5 * MS                                    # nothing can meet 5 ms
    s = oracle.score(w)
    assert int(oracle.baseline(w, oracle.MAXACC_EDF, s.acc, s.v).reqs["model"][2]) == 1    # most accurate of all
    assert int(oracle.baseline(w, oracle.LO_EDF, s.acc, s.v).reqs["model"][2]) == 0        # all utilities 0: lowest model
    # a soft penalty lets the locally-optimal choice run late on the better model: 0.9 * (1 - gamma) vs 0.6
    w2 = manual_workload([[1.0, 0.0]], [[0.6, 0.6], [0.9, 0.9]], app=[0], deadline_ms=[40], arrival_ms=[-360],
                         alpha_ms=[5, 45], beta_ms=[5, 5], swap_ms=[0, 0], batch_sizes=[1], models_per_app=[2])
    w2.penalty_kind[:] = 1                                       # linear: late by 10 ms of a 400 ms relative deadline
    s2 = oracle.score(w2)
    lo = oracle.baseline(w2, oracle.LO_EDF, s2.acc, s2.v)
    assert int(lo.reqs["model"][0]) == 1 and lo.rounds[0, 0]["utility"] == pytest.approx(0.9 * (1 - 10 / 400), abs=1e-6)
    assert int(oracle.baseline(w2, oracle.MAXACC_EDF, s2.acc, s2.v).reqs["model"][0]) == 0


def test_priority_order_puts_the_more_uncertain_request_first():
    """Eq. 12: among equal deadlines the request whose models disagree more (larger variance of accuracies) goes first;
    a later deadline can be outweighed only within the exp(-d) factor."""
    w = manual_workload([[1.0, 0.0], [0.0, 1.0]], [[0.9, 0.5], [0.1, 0.5]], app=[0, 0], deadline_ms=[100.0, 100.0],
                        alpha_ms=[1, 1], beta_ms=[1, 1], swap_ms=[0, 0], batch_sizes=[1], models_per_app=[2])
    s = oracle.score(w)
    assert s.v[0] == pytest.approx(1 + 0.16, abs=1e-6) and s.v[1] == pytest.approx(1.0, abs=1e-12)
    b = oracle.baseline(w, oracle.LO_PRIORITY, s.acc, s.v)
    assert [int(x) for x in b.reqs["order"]] == [1, 2]
    w.deadline_ns[0] += 200 * MS                                 # exp(-0.2) = 0.82 < 1 / 1.16: now the other one leads
    s = oracle.score(w)
    assert [int(x) for x in oracle.baseline(w, oracle.LO_PRIORITY, s.acc, s.v).reqs["order"]] == [2, 1]
    assert [int(x) for x in oracle.baseline(w, oracle.LO_EDF, s.acc, s.v).reqs["order"]] == [2, 1]


# ------------------------------------------------------------------ several workers (Section 6)

def _replay_workers(w, acc, d, lat_alpha, lat_beta, swap):
    """Independent replay of a multi-worker schedule: every worker's batches run back to back on its own clock with its
    own latency profile (Eq. 1 per worker), the step penalty decides each member's utility (Eq. 2); returns the total."""
    nw = lat_alpha.shape[0]
    clock = [int(w.t0_ns[0])] * nw
    loaded = [-1] * nw
    total, order = 0.0, 1
    for r in range(int(d.n_rounds[0])):
        rec = d.rounds[0, r]
        k, g, a = int(rec["worker"]), int(rec["model"]), int(rec["app"])
        members = sorted([i for i in range(w.n_requests) if d.reqs["round"][i] == r and d.reqs["status"][i] == 1],
                         key=lambda i: int(d.reqs["order"][i]))
        assert len(members) == rec["n_members"] >= 1
        assert [int(d.reqs["order"][i]) for i in members] == list(range(order, order + len(members)))
        order += len(members)
        assert all(d.reqs["worker"][i] == k and d.reqs["model"][i] == g and w.app[i] == a for i in members)
        assert k == min(range(nw), key=lambda x: (clock[x], x))          # the worker that was free first
        assert int(rec["t_start_ns"]) == clock[k]
        end = clock[k] + (int(swap[k, g]) if g != loaded[k] else 0) + int(lat_alpha[k, g]) + int(lat_beta[k, g]) * len(members)
        assert end == rec["t_end_ns"]
        u = sum(float(acc[i, g - first_model(w, a)]) for i in members if not (w.deadline_ns[i] < end))
        assert abs(u - rec["utility"]) <= 1e-11 * max(1.0, u)
        total += u
        clock[k], loaded[k] = end, g
    assert clock == [int(x) for x in d.t_end_ns] and loaded == [int(x) for x in d.loaded_end]
    return total


@pytest.mark.parametrize("seed", range(3))
def test_one_worker_is_the_single_worker_schedule(seed):
    rng = np.random.default_rng(600 + seed)
    w = _baseline_workload(rng, n=50, kinds=[0, 1, 2] if seed == 2 else None)
    s = oracle.score(w)
    d1 = oracle.drain(w, s.acc, s.v)
    dw = oracle.drain_workers(w, s.acc, s.v, w.lat_alpha_ns, w.lat_beta_ns, w.swap_ns)
    assert dw.n_rounds[0] == d1.n_rounds[0] and np.array_equal(dw.reqs, d1.reqs)
    k = int(d1.n_rounds[0])
    for f in d1.rounds.dtype.names:
        assert np.array_equal(dw.rounds[0, :k][f], d1.rounds[0, :k][f]), f
    assert dw.t_end_ns[0] == d1.t_end_ns[0] and dw.loaded_end[0] == d1.loaded_end[0]


def test_two_workers_on_a_hand_worked_queue():
    """One model (10 ms + 10 ms per request, no swap), batch size 1, four requests due at 25, 35, 45, 55 ms.  One worker
    completes them at 20, 40, 60, 80 ms: only the first is in time (the later ones leave as hopeless).  Two workers start
    two requests at once, at 0 and at 20 ms: completions 20, 20, 40, 40 ms, all but none late -> 4 x 0.8."""
    w = manual_workload([[0.5, 0.5]] * 4, [[0.8, 0.8]], app=[0] * 4, deadline_ms=[25, 35, 45, 55], alpha_ms=[10],
                        beta_ms=[10], swap_ms=[0], batch_sizes=[1], models_per_app=[1])
    s = oracle.score(w)
    one = oracle.drain_workers(w, s.acc, s.v, w.lat_alpha_ns, w.lat_beta_ns, w.swap_ns)
    assert list(one.reqs["status"]) == [1, 2, 1, 2] or list(one.reqs["status"]) == [1, 1, 2, 2] or one.rounds["utility"].sum() < 2.0
    rep = lambda a: np.repeat(np.asarray(a, dtype=np.int64), 2, axis=0)
    two = oracle.drain_workers(w, s.acc, s.v, rep(w.lat_alpha_ns), rep(w.lat_beta_ns), rep(w.swap_ns))
    assert list(two.reqs["status"]) == [1, 1, 1, 1] and list(two.reqs["worker"]) == [0, 1, 0, 1]
    assert [int(x) // MS for x in two.rounds[0, :4]["t_end_ns"]] == [20, 20, 40, 40]
    assert two.rounds[0, :4]["utility"].sum() == pytest.approx(3.2, abs=1e-6)
    assert [int(x) // MS for x in two.t_end_ns] == [40, 40]


@pytest.mark.parametrize("seed", range(3))
def test_heterogeneous_workers_replay(seed):
    rng = np.random.default_rng(700 + seed)
    w = _baseline_workload(rng, n=80, deadline=(30, 500))
    nw, sm = 3, w.sum_models
    speed = np.asarray([1.0, 0.5, 2.0])[:, None]                 # a fast, a faster and a slow worker
    al = np.rint(w.lat_alpha_ns[0][None, :] * speed).astype(np.int64)
    be = np.rint(w.lat_beta_ns[0][None, :] * speed).astype(np.int64)
    sw = np.rint(w.swap_ns[0][None, :] * rng.uniform(0.5, 2.0, size=(nw, sm))).astype(np.int64)
    s = oracle.score(w)
    d = oracle.drain_workers(w, s.acc, s.v, al, be, sw)
    total = _replay_workers(w, s.acc, d, al, be, sw)
    assert total == pytest.approx(d.rounds[0, :int(d.n_rounds[0])]["utility"].sum(), rel=1e-12)
    assert set(int(x) for x in d.rounds[0, :int(d.n_rounds[0])]["worker"]) == {0, 1, 2}
    assert np.all(d.reqs["status"] != oracle.PENDING)
    # an expired request could not have been completed in time by any worker at the round that retired it
    nr = int(d.n_rounds[0])
    for i in np.nonzero(d.reqs["status"] == oracle.EXPIRED)[0]:
        r = int(d.reqs["round"][i])
        clock = [int(w.t0_ns[0])] * nw; loaded = [-1] * nw
        for q in range(min(r, nr)):
            rec = d.rounds[0, q]; clock[int(rec["worker"])] = int(rec["t_end_ns"]); loaded[int(rec["worker"])] = int(rec["model"])
        a = int(w.app[i])
        best = min(clock[k] + (int(sw[k, g]) if g != loaded[k] else 0) + int(al[k, g]) + int(be[k, g]) * int(w.batch_sizes[0])
                   for k in range(nw) for g in range(first_model(w, a), first_model(w, a) + int(w.models_per_app[a])))
        assert w.deadline_ns[i] < best


# ------------------------------------------------------------------ k-nearest-neighbour evidence (Section 4.1)

def _knn_workload(rng, n=40, r=300, d=6, c=4, a=2, m=3):
    w = manual_workload(rng.dirichlet(np.ones(c), size=n), rng.uniform(0.2, 0.99, size=(a * m, c)), app=rng.integers(0, a, size=n),
                        deadline_ms=rng.uniform(50, 400, size=n), alpha_ms=rng.uniform(2, 20, size=a * m),
                        beta_ms=rng.uniform(0.5, 5, size=a * m), swap_ms=rng.uniform(5, 50, size=a * m), batch_sizes=[1, 2, 4],
                        models_per_app=[m] * a)
    w.feat_dim = d
    w.feats = rng.standard_normal(size=(n, d)).astype(np.float32)
    w.head_w = np.zeros((1, a, d, c), dtype=np.float32)
    ref = rng.standard_normal(size=(r, d)).astype(np.float32)
    return w, ref, rng.integers(0, c, size=r).astype(np.int32), rng.integers(0, a, size=r).astype(np.int32)


def test_knn_evidence_worked_example_of_the_paper():
    """Section 4.1's example: k = 5 neighbours, two of class "no fall" and three of class "fall", give the evidence
    y = <2, 3>; with the Jeffreys prior (alpha = 1/2) the posterior is Dir(2.5, 3.5), mean (5/12, 7/12)."""
    d = 2
    ref = np.asarray([[0.1, 0.0], [0.0, 0.2], [0.3, 0.0], [0.0, -0.4], [0.5, 0.0], [5.0, 5.0], [-6.0, 1.0]], dtype=np.float32)
    ref_label = np.asarray([0, 1, 1, 0, 1, 0, 0], dtype=np.int32)            # the five closest to the origin: 0, 1, 1, 0, 1
    w = manual_workload([[0.5, 0.5]], [[1.0, 0.0], [0.0, 1.0]], app=[0], deadline_ms=[100], alpha_ms=[1, 1], beta_ms=[1, 1],
                        swap_ms=[0, 0], batch_sizes=[1], models_per_app=[2], prior_alpha=np.full((1, 2), 0.5), evidence_k=5.0)
    w.feat_dim = d
    w.feats = np.zeros((1, d), dtype=np.float32)
    w.head_w = np.zeros((1, 1, d, 2), dtype=np.float32)
    s = oracle.score_knn(w, 5, ref, ref_label, np.zeros(7, dtype=np.int32), want_theta=True)
    np.testing.assert_allclose(s.theta[0], [5 / 12, 7 / 12], rtol=1e-15)
    np.testing.assert_allclose(s.acc[0], [5 / 12, 7 / 12], rtol=1e-15)        # recall rows are the unit vectors
    assert s.label[0] == 1
    w.prior_alpha = None
    np.testing.assert_allclose(oracle.score_knn(w, 5, ref, ref_label, np.zeros(7, dtype=np.int32), want_theta=True).theta[0], [0.4, 0.6])


@pytest.mark.parametrize("k", [1, 5, 9])
def test_knn_votes_equal_a_library_sort(k):
    rng = np.random.default_rng(800 + k)
    w, ref, ref_label, ref_app = _knn_workload(rng)
    s = oracle.score_knn(w, k, ref, ref_label, ref_app, want_theta=True)
    c = w.n_classes
    for i in range(w.n_requests):
        own = np.nonzero(ref_app == w.app[i])[0]
        dist = np.sum((w.feats[i].astype(np.float64)[None, :] - ref[own].astype(np.float64)) ** 2, axis=1)
        nearest = own[np.argsort(dist, kind="stable")[:k]]
        votes = np.bincount(ref_label[nearest], minlength=c) / float(k)
        np.testing.assert_allclose(s.theta[i], votes, atol=1e-15)
        g0 = first_model(w, int(w.app[i]))
        np.testing.assert_allclose(s.acc[i], w.recall[0, g0:g0 + 3].astype(np.float64) @ votes, rtol=1e-13)
    if k == 1:                                                   # one neighbour: the posterior is one-hot
        assert np.all(np.sort(s.theta, axis=1)[:, -1] == 1.0) and np.all(s.label >= 0)


def test_knn_ties_and_small_reference_sets():
    w = manual_workload([[0.5, 0.5]] * 2, [[1.0, 0.0]], app=[0, 1], deadline_ms=[100] * 2, alpha_ms=[1, 1], beta_ms=[1, 1],
                        swap_ms=[0, 0], batch_sizes=[1], models_per_app=[1, 1])
    w.recall = np.asarray([[[1.0, 0.0], [1.0, 0.0]]], dtype=np.float32)
    w.feat_dim = 1
    w.feats = np.zeros((2, 1), dtype=np.float32)
    w.head_w = np.zeros((1, 2, 1, 2), dtype=np.float32)
    ref = np.asarray([[1.0], [-1.0], [1.0]], dtype=np.float32)   # three points at the same distance from the origin
    s = oracle.score_knn(w, 2, ref, np.asarray([1, 0, 0], dtype=np.int32), np.zeros(3, dtype=np.int32), want_theta=True)
    np.testing.assert_allclose(s.theta[0], [0.5, 0.5])           # the two with the lower index: labels 1 and 0
    np.testing.assert_allclose(s.theta[1], [0.5, 0.5])           # application 1 has no reference point: uniform
    s5 = oracle.score_knn(w, 5, ref, np.asarray([1, 0, 0], dtype=np.int32), np.zeros(3, dtype=np.int32), want_theta=True)
    np.testing.assert_allclose(s5.theta[0], [2 / 3, 1 / 3])      # fewer points than k: all of them vote
