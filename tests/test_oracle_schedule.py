"""Pins of the oracle's scheduling rounds: invariants, replay of Eq. 1-3, Algorithm 1, brute force."""
import math

import numpy as np
import pytest

from oracle import oracle
from paper_2505_06641_b200 import synth
from helpers import (MS, brute_force_request_level, first_model, manual_workload, one_instance,
                     replay_schedule)


def _run(w, **kw):
    s = oracle.score(w)
    return s, oracle.drain(w, s.acc, s.v, **kw)


def _uniform_probs(n, c=2):
    return [[1.0 / c] * c] * n


# ------------------------------------------------------------------ utility invariants (Eq. 2)

def test_slack_deadlines_utility_is_sum_of_accuracy():
    """If every deadline is met the utility is just the accuracy of the selected model."""
    rec = [[0.6, 0.6], [0.9, 0.9]]
    w = manual_workload(_uniform_probs(4), rec, app=[0] * 4, deadline_ms=[1e5] * 4, alpha_ms=[5, 50],
                        beta_ms=[1, 10], swap_ms=[100, 300], batch_sizes=[4], models_per_app=[2])
    s, d = _run(w)
    assert d.n_rounds[0] == 1
    r = d.rounds[0, 0]
    assert r["model"] == 1 and r["n_members"] == 4 and r["n_expired"] == 0
    assert abs(r["utility"] - 4 * np.float32(0.9)) < 1e-12
    assert r["t_end_ns"] == (300 + 50 + 4 * 10) * MS
    assert list(d.reqs["order"]) == [1, 2, 3, 4] and set(d.reqs["status"]) == {oracle.SCHEDULED}


def test_late_member_contributes_exactly_zero():
    """Step penalty: a member that completes after its deadline adds nothing."""
    rec = [[0.8, 0.8]]
    # one model, l(b) = 10 + 10 b ms.  b=1 ends at 20 ms (utility 0.8); b=3 ends at 40 ms: the first
    # member (deadline 25 ms) is late and adds 0, the other two are met => 1.6, which wins.
    w = manual_workload(_uniform_probs(3), rec, app=[0] * 3, deadline_ms=[25, 40, 40], alpha_ms=[10], beta_ms=[10],
                        swap_ms=[0], batch_sizes=[1, 3], models_per_app=[1])
    s, d = _run(w)
    r = d.rounds[0, 0]
    assert d.n_rounds[0] == 1 and r["batch"] == 3 and r["n_members"] == 3 and r["n_expired"] == 0
    assert abs(r["utility"] - 2 * np.float32(0.8)) < 1e-12
    assert abs(r["util_margin"] - 0.5) < 1e-12
    # a deadline one ns before the completion time is late, one equal to it is met
    w.deadline_ns = np.asarray([25 * MS, 40 * MS - 1, 40 * MS], dtype=np.int64)
    s, d = _run(w)
    assert abs(d.rounds[0, 0]["utility"] - np.float32(0.8)) < 1e-12 and d.rounds[0, 0]["batch"] == 1
    # batch size 2 only: the earliest completion is 30 ms, so the 25 ms request can never be served
    w.deadline_ns = np.asarray([25 * MS, 40 * MS, 40 * MS], dtype=np.int64)
    w.batch_sizes = np.asarray([2], dtype=np.int32)
    s, d = _run(w)
    assert d.reqs["status"][0] == oracle.EXPIRED and d.rounds[0, 0]["n_expired"] == 1


def test_infeasible_deadlines_expire_with_zero_utility():
    w = synth.make_workload("C2")
    s, d = _run(w)
    hopeless = w.deadline_ns < w.t0_ns[0]
    assert hopeless.sum() >= int(0.3 * w.n_requests)
    assert np.all(d.reqs["status"][hopeless] == oracle.EXPIRED)
    assert np.all(d.reqs["round"][hopeless] == 0) and np.all(d.reqs["order"][hopeless] == 0)
    assert set(np.unique(d.reqs["status"])) <= {oracle.SCHEDULED, oracle.EXPIRED}


def test_chosen_utility_is_monotone_in_accuracy():
    w = synth.make_workload("C1")
    s = oracle.score(w)
    base = oracle.drain(w, s.acc, s.v, max_rounds=1, cap=1).rounds[0, 0]
    rng = np.random.default_rng(3)
    for _ in range(25):
        acc = s.acc.copy()
        i, j = rng.integers(0, w.n_requests), rng.integers(0, w.max_models)
        acc[i, j] += 0.05
        r = oracle.drain(w, acc, s.v, max_rounds=1, cap=1).rounds[0, 0]
        if r["app"] == base["app"]:
            assert r["utility"] >= base["utility"] - 1e-15


# ------------------------------------------------------------------ replay of Eq. 1-3 over emitted schedules

@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {}), ("C3", dict(n_requests=1500)),
                                     ("C5", dict(n_requests=6000))])
def test_replay_reproduces_clock_and_utility(name, kw):
    w = synth.make_workload(name, **kw)
    s, d = _run(w)
    nr = int(d.n_rounds[0])
    total = replay_schedule(w, s.acc, d.reqs, d.rounds[0], nr)
    assert abs(total - d.rounds[0, :nr]["utility"].sum()) < 1e-9
    assert np.all(d.reqs["status"] != oracle.PENDING)
    assert d.rounds[0, :nr]["n_expired"].sum() + np.sum(d.reqs["round"] == nr) == np.sum(d.reqs["status"] == oracle.EXPIRED)
    assert d.rounds[0, :nr]["n_members"].sum() == np.sum(d.reqs["status"] == oracle.SCHEDULED)


def test_replay_batched_instances():
    w = synth.make_workload("C4", n_instances=6)
    s, d = _run(w)
    for k in range(6):
        replay_schedule(w, s.acc, d.reqs, d.rounds[k], int(d.n_rounds[k]), inst=k)
        wk = one_instance(w, k)                     # an instance run alone gives the same schedule
        sk, dk = _run(wk)
        sel = w.instance == k
        assert np.array_equal(dk.reqs, d.reqs[sel]) and dk.n_rounds[0] == d.n_rounds[k]


def test_expired_requests_were_hopeless():
    """A retired request could not have met its deadline under any candidate of its application."""
    w = synth.make_workload("C1")
    s, d = _run(w)
    nr = int(d.n_rounds[0])
    al, be, sw = w.lat_alpha_ns[0], w.lat_beta_ns[0], w.swap_ns[0]
    for i in np.nonzero(d.reqs["status"] == oracle.EXPIRED)[0]:
        r = int(d.reqs["round"][i])
        t = int(d.rounds[0, r]["t_start_ns"]) if r < nr else int(d.t_end_ns[0])
        loaded = -1 if r == 0 else int(d.rounds[0, r - 1]["model"])
        a = int(w.app[i])
        best = min(t + (int(sw[g]) if g != loaded else 0) + int(al[g]) + int(be[g]) * int(w.batch_sizes[0])
                   for g in range(first_model(w, a), first_model(w, a) + int(w.models_per_app[a])))
        assert w.deadline_ns[i] < best


# ------------------------------------------------------------------ Algorithm 1 when every group fits one batch

@pytest.mark.parametrize("seed", range(6))
def test_one_batch_groups_are_served_by_eq14_order_with_eq13_models(seed):
    """With one allowed batch size that holds any group and nothing to retire, every application is served whole in
    one round.  The emitted schedule must then have the properties Algorithm 1's greedy branch is defined by: groups
    go in descending Eq. 14 priority (a common clock shift rescales all priorities alike, so the order at the
    starting clock is the order throughout), and each group runs on the model that maximises its members' summed
    Eq. 2 utility at the moment the group starts (Eq. 13 on the group; ties to the lowest model)."""
    rng = np.random.default_rng(100 + seed)
    n, a, m, c = 18, 3, 3, 4
    probs = rng.dirichlet(np.ones(c), size=n)
    w = manual_workload(probs, rng.uniform(0.3, 0.99, size=(a * m, c)), app=rng.integers(0, a, size=n),
                        deadline_ms=rng.uniform(2000, 9000, size=n), alpha_ms=rng.uniform(2, 20, size=a * m),
                        beta_ms=rng.uniform(0.5, 5, size=a * m), swap_ms=rng.uniform(50, 500, size=a * m),
                        batch_sizes=[64], models_per_app=[m] * a)
    s, d = _run(w)
    assert np.all(d.reqs["status"] == oracle.SCHEDULED)
    apps_present = sorted(set(int(x) for x in w.app))
    nr = int(d.n_rounds[0])
    rounds = d.rounds[0, :nr]
    assert sorted(int(x) for x in rounds["app"]) == apps_present           # one round per group
    t0 = int(w.t0_ns[0])
    prio = {g: float(np.mean([s.v[i] * math.exp(-(int(w.deadline_ns[i]) - t0) * 1e-9 / w.prio_time_scale_s)
                              for i in range(n) if w.app[i] == g])) for g in apps_present}
    assert [int(x) for x in rounds["app"]] == sorted(apps_present, key=lambda g: (-prio[g], g))
    prev = -1
    for r in rounds:
        g_app = int(r["app"])
        members = [i for i in range(n) if w.app[i] == g_app]
        assert r["n_members"] == len(members)
        utils = []
        for j in range(m):
            g = first_model(w, g_app) + j
            e = int(r["t_start_ns"]) + (int(w.swap_ns[0, g]) if g != prev else 0) + int(w.lat_alpha_ns[0, g]) \
                + int(w.lat_beta_ns[0, g]) * len(members)
            utils.append(sum(s.acc[i, j] for i in members if not (w.deadline_ns[i] < e)))
        assert int(r["model"]) - first_model(w, g_app) == int(np.argmax(utils))
        assert r["utility"] == pytest.approx(max(utils), rel=1e-12)
        by_key = sorted(members, key=lambda i: (int(w.deadline_ns[i]), i))
        orders = [int(d.reqs["order"][i]) for i in by_key]
        assert orders == list(range(orders[0], orders[0] + len(members)))
        prev = int(r["model"])


# ------------------------------------------------------------------ brute force on tiny queues

def test_request_level_enumerator_counts_n_factorial_m_to_the_n():
    """Section 3.1: n requests of one application have n! |M|^n candidate solutions."""
    rng = np.random.default_rng(5)
    n, m = 4, 2
    w = manual_workload(rng.dirichlet(np.ones(3), size=n), rng.uniform(0.3, 0.99, size=(m, 3)), app=[0] * n,
                        deadline_ms=rng.uniform(10, 60, size=n), alpha_ms=[4, 9], beta_ms=[1, 2], swap_ms=[5, 8],
                        batch_sizes=[1], models_per_app=[m])
    s, d = _run(w)
    best, count = brute_force_request_level(w, s.acc)
    assert count == math.factorial(n) * m ** n
    greedy = d.rounds[0, :int(d.n_rounds[0])]["utility"].sum()
    assert greedy <= best + 1e-12


@pytest.mark.parametrize("seed", range(8))
def test_greedy_never_beats_the_exhaustive_optimum(seed):
    rng = np.random.default_rng(200 + seed)
    n, apps, m = 5, 2, 2
    w = manual_workload(rng.dirichlet(np.ones(3), size=n), rng.uniform(0.3, 0.99, size=(apps * m, 3)),
                        app=rng.integers(0, apps, size=n), deadline_ms=rng.uniform(10, 80, size=n),
                        alpha_ms=rng.uniform(2, 10, size=apps * m), beta_ms=rng.uniform(1, 4, size=apps * m),
                        swap_ms=rng.uniform(2, 12, size=apps * m), batch_sizes=[1], models_per_app=[m] * apps)
    s, d = _run(w)
    best, _ = brute_force_request_level(w, s.acc)
    greedy = d.rounds[0, :int(d.n_rounds[0])]["utility"].sum()
    assert greedy <= best + 1e-12
    assert abs(replay_schedule(w, s.acc, d.reqs, d.rounds[0], int(d.n_rounds[0])) - greedy) < 1e-12


def test_greedy_is_optimal_on_a_one_model_slack_queue():
    rng = np.random.default_rng(9)
    n = 5
    w = manual_workload(rng.dirichlet(np.ones(3), size=n), rng.uniform(0.3, 0.99, size=(1, 3)), app=[0] * n,
                        deadline_ms=[1e4] * n, alpha_ms=[3], beta_ms=[2], swap_ms=[7], batch_sizes=[1],
                        models_per_app=[1])
    s, d = _run(w)
    best, _ = brute_force_request_level(w, s.acc)
    assert abs(d.rounds[0, :n]["utility"].sum() - best) < 1e-12 and abs(best - s.acc[:, 0].sum()) < 1e-12


# ------------------------------------------------------------------ ties, ordering, trace mode

def test_tie_breaks_lowest_model_then_smallest_batch_then_lowest_app():
    rec = [[0.7, 0.7]] * 4                              # four identical models, two per application
    w = manual_workload(_uniform_probs(6), rec, app=[0, 1, 0, 1, 0, 1], deadline_ms=[500] * 6, alpha_ms=[5] * 4,
                        beta_ms=[1] * 4, swap_ms=[9] * 4, batch_sizes=[1, 2, 4, 8], models_per_app=[2, 2])
    s, d = _run(w)
    r0, r1 = d.rounds[0, 0], d.rounds[0, 1]
    assert (r0["app"], r0["model"], r0["batch"], r0["n_members"]) == (0, 0, 4, 3)   # 4 and 8 both take all 3
    assert (r1["app"], r1["model"], r1["batch"], r1["n_members"]) == (1, 2, 4, 3)
    assert r0["prio_margin"] == np.inf or r0["prio_margin"] >= 0
    assert [int(x) for x in d.reqs["order"]] == [1, 4, 2, 5, 3, 6]                  # equal deadlines: id order


def test_members_follow_deadline_then_id():
    w = manual_workload(_uniform_probs(5), [[0.8, 0.8]], app=[0] * 5, deadline_ms=[900, 300, 600, 300, 100],
                        alpha_ms=[1], beta_ms=[1], swap_ms=[0], batch_sizes=[8], models_per_app=[1])
    s, d = _run(w)
    assert [int(x) for x in d.reqs["order"]] == [5, 2, 4, 3, 1]


def test_trace_mode_joins_on_arrival_and_idles_to_next_arrival():
    w = manual_workload(_uniform_probs(3), [[0.8, 0.8]], app=[0] * 3, deadline_ms=[100, 130, 1100],
                        arrival_ms=[0, 5, 1000], alpha_ms=[10], beta_ms=[10], swap_ms=[0], batch_sizes=[1, 2],
                        models_per_app=[1], trace_mode=True)
    s, d = _run(w)
    r = d.rounds[0, :int(d.n_rounds[0])]
    # t=0: only request 0 is there (20 ms); t=20: request 1 (20 ms); then idle until 1000 ms
    assert [int(x) for x in r["n_members"]] == [1, 1, 1]
    assert [int(x) // MS for x in r["t_start_ns"]] == [0, 20, 1000]
    assert [int(x) // MS for x in r["t_end_ns"]] == [20, 40, 1020]
    snap = oracle.drain(w, s.acc, s.v, trace_mode=False)                  # snapshot: everything is pending at t0
    assert int(snap.rounds[0, 0]["n_members"]) == 2


def test_group_priority_value_and_choice():
    """Eq. 14 over Eq. 12 by hand: group 0 has the later deadline but the larger accuracy variance."""
    rec = [[0.1, 0.1], [0.9, 0.9], [0.5, 0.5], [0.5, 0.5]]
    w = manual_workload(_uniform_probs(2), rec, app=[0, 1], deadline_ms=[1100, 1000], alpha_ms=[1] * 4, beta_ms=[1] * 4,
                        swap_ms=[0] * 4, batch_sizes=[1], models_per_app=[2, 2])
    s, d = _run(w)
    p0 = (1 + 0.16) * math.exp(-1.1)
    p1 = 1.0 * math.exp(-1.0)
    assert p0 > p1 and d.rounds[0, 0]["app"] == 0
    assert abs(d.rounds[0, 0]["group_priority"] - p0) < 1e-7
    assert abs(d.rounds[0, 0]["prio_margin"] - (p0 - p1) / p0) < 1e-6


def test_max_rounds_stops_early_and_leaves_the_rest_pending():
    w = synth.make_workload("C2")
    s = oracle.score(w)
    d = oracle.drain(w, s.acc, s.v, max_rounds=2)
    full = oracle.drain(w, s.acc, s.v)
    assert d.n_rounds[0] == 2 and np.array_equal(d.rounds[0, :2], full.rounds[0, :2])
    assert np.sum(d.reqs["status"] == oracle.PENDING) > 0


def test_short_circuit_candidate_is_static_and_wins_when_nothing_else_is_in_time():
    """Section 4.3: the SneakPeek model as one more candidate with zero latency and its profiled (static) accuracy.
    In the profile format it is a recall row with one value for every label, so Eq. 9 gives that value for every
    request; with deadlines that no real variant can meet it is the only candidate with non-zero utility."""
    from oracle import oracle
    from paper_2505_06641_b200 import synth
    w = synth.with_short_circuit(synth.make_workload("C1", n_requests=60), [0.55, 0.6, 0.65])
    assert list(w.models_per_app) == [5, 5, 5] and w.recall.shape[1] == 15
    s = oracle.score(w)
    for a in range(3):
        np.testing.assert_allclose(s.acc[w.app == a, 4], [0.55, 0.6, 0.65][a], rtol=1e-6)
    # every deadline 1 ms after the starting clock: real variants need at least 2.5 ms
    w.deadline_ns = np.full_like(w.deadline_ns, int(w.t0_ns[0]) + synth.MS)
    d = oracle.drain(w, s.acc, s.v)
    assert np.all(d.reqs["status"] == 1)
    first = np.concatenate([[0], np.cumsum(w.models_per_app)])
    assert np.all(d.reqs["model"] == first[w.app + 1] - 1)            # the short-circuit variant of its application
    nr = int(d.n_rounds[0])
    assert np.all(d.rounds[0, :nr]["t_end_ns"] == w.t0_ns[0])           # zero latency: the clock does not move
    np.testing.assert_allclose(d.rounds[0, :nr]["utility"].sum(), s.acc[np.arange(60), 4].astype(np.float64).sum(), rtol=1e-12)


@pytest.mark.parametrize("kind", [1, 2])
def test_soft_penalty_late_member_keeps_part_of_its_accuracy(kind):
    """One request, one variant, completion late by a quarter of the relative deadline: Eq. 2 leaves
    acc * (1 - gamma), gamma = 1/4 (linear) or 1/28 (sigmoid: 1 / (1 + 3^3)); late by all of it: retired."""
    from oracle import oracle
    w = manual_workload([[0.5, 0.5]], [[0.8, 0.8]], app=[0], deadline_ms=[40], arrival_ms=[0], alpha_ms=[40], beta_ms=[10],
                        swap_ms=[0], batch_sizes=[1], models_per_app=[1])
    w.penalty_kind = np.asarray([kind], dtype=np.int32)
    s = oracle.score(w)
    d = oracle.drain(w, s.acc, s.v)                       # completes at 50 ms: 10 ms late, relative deadline 40 ms
    assert d.reqs["status"][0] == 1
    gamma = 0.25 if kind == 1 else 1.0 / 28.0
    np.testing.assert_allclose(d.rounds[0, 0]["utility"], s.acc[0, 0] * (1.0 - gamma), rtol=1e-12)
    assert abs(s.acc[0, 0] - 0.8) < 1e-7
    w.lat_alpha_ns = np.asarray([[70 * 1_000_000]], dtype=np.int64)      # completes at 80 ms: late by the whole 40 ms
    d = oracle.drain(w, s.acc, s.v)
    assert d.reqs["status"][0] == 2 and d.n_rounds[0] == 0


@pytest.mark.parametrize("kind", [1, 2])
def test_soft_penalties_replay_and_never_below_the_step_schedule(kind):
    from oracle import oracle
    w = synth.make_workload("C1")
    s = oracle.score(w)
    step = oracle.drain(w, s.acc, s.v)
    w.penalty_kind = np.full(3, kind, dtype=np.int32)
    d = oracle.drain(w, s.acc, s.v)
    nr = int(d.n_rounds[0])
    total = replay_schedule(w, s.acc, d.reqs, d.rounds[0], nr)
    np.testing.assert_allclose(total, d.rounds[0, :nr]["utility"].sum(), rtol=1e-12)
    # a softer penalty retires fewer requests at the head of the queues
    assert (d.reqs["status"] == 2).sum() <= (step.reqs["status"] == 2).sum()
