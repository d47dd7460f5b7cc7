"""Parity of the CUDA library with the CPU oracle, element by element (needs a B200; run with -m gpu)."""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth
from helpers import manual_workload
from parity import ACC_RTOL, check_schedule, check_scores

pytestmark = pytest.mark.gpu


def _both(w, guards=None, **kw):
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v, **{k: v for k, v in kw.items() if k in ("max_rounds", "cap")})
    ses = runner.Session(w)
    if guards is not None:
        api.sp_set_options(ses.ctx, trace_mode=bool(w.trace_mode), guard_utility=guards[0], guard_priority=guards[1])
    res = ses.run(**kw)
    ses.close()
    return s, od, res


CASES = [("C1", {}), ("C2", {}), ("C3", dict(n_requests=3000)), ("C4", dict(n_instances=40)),
         ("C5", dict(n_requests=20000)),
         ("C1", dict(n_requests=1)), ("C1", dict(n_requests=129)), ("C2", dict(n_requests=65)),
         ("C4", dict(n_instances=3, n_requests=131)), ("C3", dict(n_requests=70, models=5)),
         ("C2", dict(n_requests=20000)), ("C2", dict(n_requests=70001)),     # large snapshots: sorted by the whole GPU
         # many instances per block with 2 and 1 feature slabs per tile: the head operand is rebuilt at every instance
         # change while tiles of the previous instance may still be in the tensor pipe
         ("C4", dict(n_instances=700, feat_dim=64)), ("C4", dict(n_instances=700, n_requests=300, feat_dim=32))]


@pytest.mark.parametrize("name,kw", CASES)
def test_scores_and_schedule_match_oracle(name, kw):
    w = synth.make_workload(name, **kw)
    s, od, res = _both(w)
    worst = check_scores(res, s)
    skipped = check_schedule(w, res, od)
    assert skipped == 0, "unexpected near-tie in a seeded case"
    assert worst < ACC_RTOL


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {}), ("C4", dict(n_instances=12)),
                                     ("C5", dict(n_requests=4000)), ("C3", dict(n_requests=400))])
def test_fp64_reevaluation_path_gives_the_same_schedule(name, kw):
    """Guards of 1.0 send every round through the fp64 re-scoring; the schedule must not change."""
    w = synth.make_workload(name, **kw)
    s, od, res = _both(w, guards=(1.0, 1.0))
    check_schedule(w, res, od)
    nr = int(res.n_rounds.sum())
    assert res.stats["exact_utility"] > 0 and res.stats["exact_rows"] > 0
    multi = res.rounds["exact"][res.rounds["n_members"] > 0]
    assert np.all(multi & 2 | (multi == 0) | (multi & 1)) and nr == res.stats["rounds"]
    # utilities decided in fp64 agree with the oracle to rounding
    for k in range(int(w.n_instances)):
        n = int(od.n_rounds[k])
        ex = (res.rounds[k, :n]["exact"] & 2) != 0
        np.testing.assert_allclose(res.rounds[k, :n]["utility"][ex], od.rounds[k, :n]["utility"][ex], rtol=1e-12)


def test_dirichlet_prior_and_ragged_model_sets():
    rng = np.random.default_rng(11)
    n, c = 200, 7
    w = manual_workload(rng.dirichlet(np.ones(c), size=n), rng.uniform(0.2, 0.99, size=(6, c)),
                        app=rng.integers(0, 3, size=n), deadline_ms=rng.uniform(50, 900, size=n),
                        alpha_ms=rng.uniform(2, 20, size=6), beta_ms=rng.uniform(0.5, 5, size=6),
                        swap_ms=rng.uniform(5, 50, size=6), batch_sizes=[1, 2, 4, 8], models_per_app=[1, 2, 3],
                        prior_alpha=np.full((3, c), 0.5), evidence_k=5.0)
    s, od, res = _both(w)
    check_scores(res, s)
    check_schedule(w, res, od)
    assert np.all(res.acc[w.app == 0, 1:] == 0) and np.all(res.v[w.app == 0] == 1.0)


def test_padded_classes_with_minus_inf_bias():
    w = synth.make_workload("C1", n_requests=100)
    w.head_b[0, 1, 6:] = -np.inf          # application 1 has only 6 labels
    w.recall[0, 4:8, 6:] = 0.0
    s, od, res = _both(w)
    check_scores(res, s)
    check_schedule(w, res, od)


def test_empty_request_set():
    from paper_2505_06641_b200 import runner
    w = synth.make_workload("C1", n_requests=1)
    for f in ("feats", "app", "arrival_ns", "deadline_ns", "instance"):
        setattr(w, f, getattr(w, f)[:0])
    ses = runner.Session(w)
    res = ses.run(max_rounds=4, cap=4)
    assert res.n_rounds[0] == 0 and len(res.reqs) == 0
    ses.close()


def test_rounds_can_be_run_in_several_calls():
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    import torch
    w = synth.make_workload("C2")
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(64); ses.score()
    got = []
    for _ in range(40):
        ses.schedule(3)
        api.sp_check(ses.ctx)
        k = int(ses.n_done.cpu()[0])
        got.append(ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE)[0, :k].copy())
        if k < 3:
            break
    got = np.concatenate(got)
    assert len(got) == od.n_rounds[0]
    for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
        assert np.array_equal(got[f], od.rounds[0, :len(got)][f]), f
    ses.close()


def test_trace_mode_idle_clock_jump():
    w = manual_workload([[0.5, 0.5]] * 3, [[0.8, 0.8]], app=[0] * 3, deadline_ms=[100, 130, 1100],
                        arrival_ms=[0, 5, 1000], alpha_ms=[10], beta_ms=[10], swap_ms=[0], batch_sizes=[1, 2],
                        models_per_app=[1], trace_mode=True)
    s, od, res = _both(w)
    check_schedule(w, res, od)
    assert [int(x) // synth.MS for x in res.rounds[0, :3]["t_start_ns"]] == [0, 20, 1000]


def test_host_buffer_entry_point_matches_device_path():
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C4", n_instances=9)
    ses = runner.Session(w)
    ref = ses.run()
    n, ni, cap = w.n_requests, w.n_instances, ref.rounds.shape[1]
    reqs = np.zeros(n, dtype=api.REQ_DTYPE)
    rounds = np.zeros((ni, cap), dtype=api.ROUND_DTYPE)
    nd = np.zeros(ni, dtype=np.int32)
    api.sp_run_host(ses.ctx, n, w.feats, w.app, w.arrival_ns, w.deadline_ns, w.instance, w.t0_ns,
                    np.full(ni, -1, dtype=np.int32), 10_000, reqs, rounds, cap, nd)
    assert np.array_equal(reqs, ref.reqs) and np.array_equal(nd, ref.n_rounds)
    for k in range(ni):
        assert np.array_equal(rounds[k, :nd[k]], ref.rounds[k, :nd[k]])
    ses.close()


def test_errors_are_reported_not_crashes():
    import torch
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C1")
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(8); ses.score()
    ses.dev["app"][5] = 77                          # out-of-range application id
    ses.score(); ses.schedule(8)
    with pytest.raises(api.SpError) as e:
        api.sp_check(ses.ctx)
    assert e.value.status == api.SP_EINVAL
    assert int(ses.n_done.cpu()[0]) == 0            # nothing was scheduled from a rejected table
    ses.dev["app"][5] = 0
    ses.score(); ses.schedule(8); api.sp_check(ses.ctx)
    assert int(ses.n_done.cpu()[0]) > 0
    w.batch_sizes = np.asarray([4, 2], dtype=np.int32)
    with pytest.raises(api.SpError) as e:
        api.sp_load_profiles(ses.ctx, w)
    assert e.value.status == api.SP_EINVAL
    ses.close()


def _drop_requests(w, keep):
    for f in ("feats", "app", "arrival_ns", "deadline_ns", "instance"):
        setattr(w, f, np.ascontiguousarray(getattr(w, f)[keep]))
    return w


def test_batched_rounds_resume_after_a_partial_call():
    """Batched mode: a call that stops after one round per instance leaves a state the next calls continue from."""
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C4", n_instances=6, n_requests=200)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(4); ses.score()
    got = [[] for _ in range(6)]
    for _ in range(64):
        ses.schedule(1)
        api.sp_check(ses.ctx)
        nd = ses.n_done.cpu().numpy()
        rr = ses.rounds.cpu().numpy().reshape(6, -1).view(api.ROUND_DTYPE)
        for k in range(6):
            got[k].extend(rr[k, :nd[k]].copy())
        if nd.sum() == 0:
            break
    for k in range(6):
        n = int(od.n_rounds[k])
        assert len(got[k]) == n
        for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
            assert [int(r[f]) for r in got[k]] == [int(x) for x in od.rounds[k, :n][f]], (k, f)
    api.sp_get_requests(ses.ctx, 0, ses.n, ses.recs)
    reqs = ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:ses.n]
    for f in ("status", "round", "model", "order"):
        assert np.array_equal(reqs[f], od.reqs[f]), f
    ses.close()


def test_batched_instances_of_very_different_sizes():
    """One instance far above the average size is left to the block-per-instance kernel in the same call."""
    w = synth.make_workload("C4", n_instances=8, n_requests=512)
    inst = np.asarray(w.instance)
    rank = np.arange(len(inst)) - np.searchsorted(inst, inst)      # position inside the instance
    keep = (inst == 3) | (rank < 40)
    w = _drop_requests(w, keep)
    s, od, res = _both(w)
    check_scores(res, s)
    check_schedule(w, res, od)


def test_full_size_batched_workload_on_sampled_instances():
    """The benchmark's own launch (16,384 instances x 512 requests in one sp_score / sp_schedule_round) checked
    against the oracle on a seeded sample of instances, each regenerated on its own from its seed."""
    from types import SimpleNamespace
    from oracle import oracle
    from paper_2505_06641_b200 import runner
    full = synth._SPECS["C4"][2]
    w = synth.make_workload("C4", n_instances=full)
    ses = runner.Session(w)
    res = ses.run(cap=16)
    ses.close()
    assert res.stats["score_kernel"] == 2                      # the tensor-core kernel is the one that ran
    inst = np.asarray(w.instance)
    starts = np.searchsorted(inst, np.arange(full + 1))
    rng = np.random.default_rng(5)
    sample = sorted(set(rng.integers(0, full, size=40).tolist()) | {0, full - 1})
    worst = 0.0
    for i in sample:
        wi = synth.make_workload("C4", n_instances=1, first_instance=i)
        sl = slice(starts[i], starts[i + 1])
        assert np.array_equal(wi.deadline_ns, w.deadline_ns[sl]) and np.array_equal(wi.feats, w.feats[sl])
        s = oracle.score(wi)
        od = oracle.drain(wi, s.acc, s.v, cap=16)
        rounds = res.rounds[i:i + 1].copy()
        rounds["instance"] = 0
        part = SimpleNamespace(acc=res.acc[sl], v=res.v[sl], reqs=res.reqs[sl], rounds=rounds,
                               n_rounds=res.n_rounds[i:i + 1], t_end_ns=res.t_end_ns[i:i + 1],
                               loaded_end=res.loaded_end[i:i + 1])
        worst = max(worst, check_scores(part, s))
        assert check_schedule(wi, part, od) == 0
    assert worst < ACC_RTOL
    # properties that hold for every instance: every request got a final record, orders are 1..#scheduled
    st = res.reqs["status"]
    assert np.all(st != 0)
    sched = st == 1
    per_inst = np.add.reduceat(sched.astype(np.int64), starts[:-1])
    max_order = np.maximum.reduceat(np.where(sched, res.reqs["order"], 0), starts[:-1])
    assert np.array_equal(per_inst, max_order)


@pytest.mark.parametrize("name,kw,tight", [("C1", {}, False), ("C4", dict(n_instances=10), False),
                                           ("C1", dict(n_requests=200), True), ("C5", dict(n_requests=3000), False)])
def test_short_circuit_candidate(name, kw, tight):
    """Section 4.3's zero-latency candidate with static accuracy, added to every application's variants."""
    w = synth.with_short_circuit(synth.make_workload(name, **kw), [0.55, 0.6, 0.65])
    if tight:                             # nothing but the zero-latency candidate can meet these deadlines
        w.deadline_ns = np.maximum(w.deadline_ns, w.t0_ns[0]) * 0 + int(w.t0_ns[0]) + synth.MS
    s, od, res = _both(w)
    check_scores(res, s)
    check_schedule(w, res, od)
    if tight:
        assert np.all(res.reqs["status"] == 1) and np.all(res.rounds[0, :int(res.n_rounds[0])]["t_end_ns"] == w.t0_ns[0])


@pytest.mark.parametrize("name,kw,kinds,guards", [
    ("C1", {}, [1, 1, 1], None), ("C1", {}, [2, 2, 2], None), ("C2", {}, [2, 0, 1], None),
    ("C4", dict(n_instances=8), [0, 1, 2], None), ("C5", dict(n_requests=6000), [2, 2, 2], None),
    ("C1", {}, [2, 1, 0], (1.0, 1.0)), ("C3", dict(n_requests=1500), [1, 2, 0], None)])
def test_linear_and_sigmoid_penalties(name, kw, kinds, guards):
    """Section 5.1's soft penalties (utility degrades after the deadline over the relative deadline), per application;
    with guards of 1.0 every decision also goes through the fp64 re-evaluation."""
    w = synth.make_workload(name, **kw)
    w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    s, od, res = _both(w, guards=guards)
    check_scores(res, s)
    check_schedule(w, res, od)
    late = od.reqs["status"] == 1
    assert late.any()


def _shape_cases():
    """Seeded draws of small shapes around the limits of the scoring kernels (labels, feature slabs, model counts)."""
    rng = np.random.default_rng(2024)
    cases = []
    for k in range(14):
        base = ["C4", "C1", "C2"][k % 3]
        kw = dict(n_apps=int(rng.integers(1, 5)), models=int(rng.integers(1, 7)),
                  n_classes=int(rng.choice([3, 5, 8, 10, 12, 16, 20, 21, 32, 40])),
                  feat_dim=int(rng.choice([32, 64, 96, 128, 160, 256])), n_requests=int(rng.integers(1, 700)))
        if base == "C4":
            kw["n_instances"] = int(rng.choice([2, 37, 400]))
            kw["n_requests"] = int(rng.integers(1, 300))
        cases.append((base, kw))
    return cases


@pytest.mark.parametrize("name,kw", _shape_cases())
def test_random_shapes_match_oracle(name, kw):
    w = synth.make_workload(name, **kw)
    s, od, res = _both(w)
    worst = check_scores(res, s)
    check_schedule(w, res, od)
    assert worst < ACC_RTOL


def test_sigmoid_penalty_that_rounds_to_one_before_the_request_is_hopeless():
    """A request late by all but a few millionths of its relative deadline has a sigmoid penalty that is 1.0 in
    fp64 although x < 1: it is not hopeless yet (the test is on the integer times) and, if served then, earns exactly
    nothing, on both sides (one of these 1,500 instances has two such requests)."""
    w = synth.make_workload("C4", n_apps=4, models=1, n_classes=24, feat_dim=128, n_requests=329, n_instances=1500)
    w.penalty_kind = np.array([0, 2, 1, 2], dtype=np.int32)
    s, od, res = _both(w)
    check_scores(res, s)
    check_schedule(w, res, od)


@pytest.mark.parametrize("name,kw", [("C4", dict(n_instances=9)), ("C1", {})])
def test_a_call_for_zero_rounds_changes_nothing(name, kw):
    """sp_schedule_round(max_rounds = 0) retires nothing and starts nothing, in batched mode as for one instance: the
    clock can still be set afterwards, and the rounds that follow are the oracle's."""
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload(name, **kw)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(600); ses.score()
    ses.schedule(0)
    api.sp_check(ses.ctx)
    api.sp_get_requests(ses.ctx, 0, ses.n, ses.recs)
    reqs = ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:ses.n]
    assert np.all(reqs["status"] == api.SP_PENDING) and int(ses.n_done.sum()) == 0
    api.sp_set_clocks(ses.ctx, ses.dev["t0"], ses.dev["l0"])
    ses.schedule(10_000)
    api.sp_check(ses.ctx)
    api.sp_get_requests(ses.ctx, 0, ses.n, ses.recs)
    reqs = ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:ses.n]
    for f in ("status", "round", "model", "order"):
        assert np.array_equal(reqs[f], od.reqs[f]), f
    assert np.array_equal(ses.n_done.cpu().numpy(), od.n_rounds)
    ses.close()


def test_zero_guards_select_the_defaults():
    """A zero-initialised options struct must not switch the fp64 re-evaluation of near-ties off."""
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C4", n_instances=300)
    ses = runner.Session(w)
    ref = ses.run()
    api.sp_set_options(ses.ctx, trace_mode=False, guard_utility=0.0, guard_priority=0.0)
    got = ses.run()
    ses.close()
    assert np.array_equal(ref.reqs, got.reqs)
    assert got.stats["exact_utility"] + got.stats["exact_priority"] == ref.stats["exact_utility"] + ref.stats["exact_priority"]


@pytest.mark.parametrize("name,kw", [("C2", dict(n_requests=20000)), ("C5", dict(n_requests=20000)),
                                     ("C3", dict(n_requests=6000, n_classes=200, feat_dim=256))])
def test_near_ties_in_one_large_instance_are_rescored_by_the_whole_gpu(name, kw):
    """Guards of 1.0 make every round a near-tie between groups, which needs the fp64 scores of every live request.  In a
    large single instance that is thousands of rows: the block stops before the round, the whole GPU scores the rows,
    and the rounds resume within the same call.  Same schedule as the oracle, and the rows are scored once."""
    w = synth.make_workload(name, **kw)
    s, od, res = _both(w, guards=(1.0, 1.0))
    check_schedule(w, res, od)
    assert res.stats["exact_priority"] > 0
    assert 0 < res.stats["exact_rows"] <= w.n_requests
