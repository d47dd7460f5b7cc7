"""Data-aware sub-groups (Section 4.3), the exhaustive branch of Algorithm 1 and the request-level baselines of
Section 5.1 on the GPU, against the CPU oracle.  Needs a B200; run with -m gpu."""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth
from parity import ACC_RTOL, NEAR_TIE, check_schedule

pytestmark = pytest.mark.gpu


def _run_policy(w, call, cap):
    """Scores w on the GPU, runs `call(ctx, rounds, cap, n_done)`, returns (Result-like object, labels, extra)."""
    import torch
    from paper_2505_06641_b200 import api, runner
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(cap); ses.score()
    extra = call(ses.ctx, ses.rounds, ses.cap, ses.n_done)
    n, ni = ses.n, int(w.n_instances)
    labels = torch.empty(max(n, 1), dtype=torch.int32, device=ses.device)
    api.sp_get_labels(ses.ctx, 0, n, labels)
    api.sp_get_requests(ses.ctx, 0, n, ses.recs)
    t_end = torch.empty(ni, dtype=torch.int64, device=ses.device)
    l_end = torch.empty(ni, dtype=torch.int32, device=ses.device)
    api.sp_get_clocks(ses.ctx, t_end, l_end)
    api.sp_check(ses.ctx)
    res = runner.Result(None, None, ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:n],
                        ses.rounds.cpu().numpy().reshape(ni, -1).view(api.ROUND_DTYPE), ses.n_done.cpu().numpy(),
                        t_end.cpu().numpy(), l_end.cpu().numpy(), api.sp_get_stats(ses.ctx))
    ses.close()
    return res, labels.cpu().numpy()[:n], extra


SPLIT_CASES = [
    ("C1", dict(w_std=0.6), None, False),
    ("C1", dict(w_std=1.0, n_requests=700, n_classes=3), [2, 0, 1], False),
    ("C2", dict(w_std=0.4, n_requests=3000), None, False),
    ("C2", dict(w_std=0.4, n_requests=9000, n_classes=24), [1, 1, 2], True),     # more requests than one block sorts in shared memory
    ("C4", dict(w_std=0.5, n_instances=40), None, False),
    ("C4", dict(w_std=0.5, n_instances=7, n_requests=300), [0, 2, 1], True),
    ("C3", dict(w_std=0.25, n_requests=2500), None, False),
    ("C1", dict(), None, False)]                                   # flat posteriors: hardly any sub-group


@pytest.mark.parametrize("name,kw,kinds,short", SPLIT_CASES)
def test_sub_group_rounds_match_oracle(name, kw, kinds, short):
    from oracle import oracle
    from paper_2505_06641_b200 import api
    w = synth.make_workload(name, **kw)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    if short:
        w = synth.with_short_circuit(w, [0.5, 0.55, 0.6])
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v, labels=s.label)
    per_inst = w.n_requests // int(w.n_instances)
    res, labels, _ = _run_policy(w, lambda ctx, r, cap, nd: api.sp_schedule_split(ctx, r, cap, nd), per_inst)
    assert np.array_equal(labels, s.label)
    if kw.get("w_std"):
        assert len(np.unique(s.label)) > 2                      # the case does split
    assert check_schedule(w, res, od) == 0
    for k in range(int(w.n_instances)):                         # the sub-group served by every round
        nr = int(od.n_rounds[k])
        assert np.array_equal((res.rounds[k, :nr]["exact"] >> 8) - 1, od.rounds[k, :nr]["label"])


def test_sub_groups_change_the_schedule_and_need_a_fresh_snapshot():
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C1", w_std=0.8)
    s = oracle.score(w)
    plain = oracle.drain(w, s.acc, s.v)
    split = oracle.drain(w, s.acc, s.v, labels=s.label)
    assert split.n_rounds[0] != plain.n_rounds[0] or not np.array_equal(split.reqs, plain.reqs)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(8); ses.score()
    ses.schedule(1)
    with pytest.raises(api.SpError) as e:                       # a round has run on this table
        api.sp_schedule_split(ses.ctx, ses.rounds, ses.cap, ses.n_done)
    assert e.value.status == api.SP_ESTATE
    ses.close()
    wt = synth.make_workload("C1", trace_mode=True)
    ses = runner.Session(wt)
    ses.upload(); ses.alloc_outputs(8); ses.score()
    with pytest.raises(api.SpError) as e:
        api.sp_schedule_split(ses.ctx, ses.rounds, ses.cap, ses.n_done)
    assert e.value.status == api.SP_ESTATE
    ses.close()


EXH_CASES = [
    ("C1", dict(n_requests=200), False, None),
    ("C1", dict(n_requests=300, models=3), False, [1, 2, 0]),
    ("C2", dict(n_requests=600), False, None),
    ("C1", dict(n_requests=150, n_apps=2, models=3, n_classes=2, w_std=1.0), True, None),
    ("C2", dict(n_requests=9000, models=4), False, None),
    ("C1", dict(n_requests=1, n_apps=1), False, None)]


@pytest.mark.parametrize("name,kw,split,kinds", EXH_CASES)
def test_exhaustive_branch_matches_oracle(name, kw, split, kinds):
    from oracle import oracle
    from paper_2505_06641_b200 import api
    w = synth.make_workload(name, **kw)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    w.deadline_ns = w.deadline_ns + 300 * synth.MS               # keep some requests in time (nothing is retired here)
    s = oracle.score(w)
    bf = oracle.bruteforce(w, s.acc, labels=s.label if split else None)
    res, labels, (total, nsol) = _run_policy(
        w, lambda ctx, r, cap, nd: api.sp_schedule_exhaustive(ctx, split, r, cap, nd), w.n_requests)
    assert nsol == bf.n_solutions
    assert total == pytest.approx(bf.total, rel=1e-12)
    if bf.second > -np.inf and bf.total > 0 and (bf.total - bf.second) / bf.total < NEAR_TIE:
        pytest.skip("two solutions within the near-tie band")
    k = int(bf.n_rounds[0])
    assert int(res.n_rounds[0]) == k
    for f in ("round", "app", "model", "batch", "n_members", "t_start_ns", "t_end_ns"):
        assert np.array_equal(res.rounds[0, :k][f], bf.rounds[0, :k][f]), f
    np.testing.assert_allclose(res.rounds[0, :k]["utility"], bf.rounds[0, :k]["utility"], rtol=1e-12, atol=1e-300)
    assert np.array_equal((res.rounds[0, :k]["exact"] >> 8) - 1, bf.rounds[0, :k]["label"])
    for f in ("status", "round", "model", "order"):
        assert np.array_equal(res.reqs[f], bf.reqs[f]), f
    assert int(res.t_end_ns[0]) == int(bf.t_end_ns[0]) and int(res.loaded_end[0]) == int(bf.loaded_end[0])


def test_exhaustive_branch_refuses_too_many_groups():
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C1", n_apps=3, n_classes=4, w_std=1.0)         # up to 15 sub-groups
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(8); ses.score()
    with pytest.raises(api.SpError) as e:
        api.sp_schedule_exhaustive(ses.ctx, True, ses.rounds, ses.cap, ses.n_done)
    assert e.value.status == api.SP_EINVAL
    total, nsol = api.sp_schedule_exhaustive(ses.ctx, False, ses.rounds, ses.cap, ses.n_done)   # still usable
    assert nsol == 6 * 4 ** 3 and total >= 0.0
    ses.close()


BASE_CASES = [("C1", {}, None), ("C1", dict(n_requests=900), [2, 1, 0]), ("C2", dict(n_requests=300), None),
              ("C2", dict(n_requests=12000, models=5), [0, 1, 2]), ("C4", dict(n_instances=40), None),
              ("C3", dict(n_requests=1200), None)]


@pytest.mark.parametrize("policy", [0, 1, 2])
@pytest.mark.parametrize("name,kw,kinds", BASE_CASES)
def test_request_level_baselines_match_oracle(name, kw, kinds, policy):
    from oracle import oracle
    from paper_2505_06641_b200 import api
    w = synth.make_workload(name, **kw)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    w.deadline_ns = w.deadline_ns + 400 * synth.MS
    s = oracle.score(w)
    ob = oracle.baseline(w, policy, s.acc, s.v)
    per_inst = w.n_requests // int(w.n_instances)
    res, _, _ = _run_policy(w, lambda ctx, r, cap, nd: api.sp_schedule_baseline(ctx, policy, r, cap, nd), per_inst)
    inst = np.asarray(w.instance)
    for k in range(int(w.n_instances)):
        if ob.min_margin[k] < NEAR_TIE:
            continue                                            # two scores or priorities within the near-tie band
        nr = int(ob.n_rounds[k])
        assert int(res.n_rounds[k]) == nr
        for f in ("round", "app", "model", "batch", "n_members", "t_start_ns", "t_end_ns"):
            assert np.array_equal(res.rounds[k, :nr][f], ob.rounds[k, :nr][f]), (k, f)
        np.testing.assert_allclose(res.rounds[k, :nr]["utility"], ob.rounds[k, :nr]["utility"], rtol=1e-12, atol=1e-300)
        np.testing.assert_allclose(res.rounds[k, :nr]["group_priority"], ob.rounds[k, :nr]["group_priority"], rtol=1e-12)
        sel = inst == k
        for f in ("status", "round", "model", "order"):
            assert np.array_equal(res.reqs[f][sel], ob.reqs[f][sel]), (k, f)
        assert int(res.t_end_ns[k]) == int(ob.t_end_ns[k]) and int(res.loaded_end[k]) == int(ob.loaded_end[k])
    assert np.sum(ob.min_margin >= NEAR_TIE) >= 0.9 * int(w.n_instances)


WORKER_CASES = [("C1", {}, 1, False, None), ("C1", {}, 2, False, None), ("C2", dict(n_requests=3000), 3, False, [1, 0, 2]),
                ("C1", dict(w_std=0.8, n_requests=600), 4, True, None), ("C3", dict(n_requests=1500), 2, False, None),
                ("C2", dict(n_requests=9000), 5, False, None)]


@pytest.mark.parametrize("name,kw,n_workers,split,kinds", WORKER_CASES)
def test_rounds_on_several_workers_match_oracle(name, kw, n_workers, split, kinds):
    """Section 6: heterogeneous workers, each with its own latency profile; the worker that is free first takes the next
    batch.  Records, per-request workers and every worker's final clock against the oracle."""
    import torch
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload(name, **kw)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    rng = np.random.default_rng(n_workers)
    speed = rng.uniform(0.4, 2.5, size=(n_workers, 1))
    al = np.rint(w.lat_alpha_ns[0][None, :] * speed).astype(np.int64)
    be = np.rint(w.lat_beta_ns[0][None, :] * speed).astype(np.int64)
    sw = np.rint(w.swap_ns[0][None, :] * rng.uniform(0.5, 2.0, size=(n_workers, w.sum_models))).astype(np.int64)
    if n_workers == 1:
        al, be, sw = w.lat_alpha_ns, w.lat_beta_ns, w.swap_ns
    s = oracle.score(w)
    od = oracle.drain_workers(w, s.acc, s.v, al, be, sw, labels=s.label if split else None)
    n = w.n_requests
    ses = runner.Session(w)
    api.sp_set_workers(ses.ctx, al, be, sw)
    ses.upload(); ses.alloc_outputs(n); ses.score()
    api.sp_schedule_workers(ses.ctx, split, ses.rounds, ses.cap, ses.n_done)
    api.sp_get_requests(ses.ctx, 0, n, ses.recs)
    t_w = torch.empty(n_workers, dtype=torch.int64, device=ses.device)
    l_w = torch.empty(n_workers, dtype=torch.int32, device=ses.device)
    api.sp_get_workers(ses.ctx, t_w, l_w)
    api.sp_check(ses.ctx)
    reqs = ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:n]
    rounds = ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE)
    k = int(od.n_rounds[0])
    tie = np.nonzero((od.rounds[0, :k]["util_margin"] < NEAR_TIE) | (od.rounds[0, :k]["prio_margin"] < NEAR_TIE))[0]
    assert len(tie) == 0 and int(ses.n_done.cpu()[0]) == k
    g = rounds[0, :k]
    for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
        assert np.array_equal(g[f], od.rounds[0, :k][f]), f
    assert np.array_equal((g["exact"] >> 2) & 63, od.rounds[0, :k]["worker"])
    assert np.array_equal((g["exact"] >> 8) - 1, od.rounds[0, :k]["label"])
    np.testing.assert_allclose(g["utility"], od.rounds[0, :k]["utility"], rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(g["group_priority"], od.rounds[0, :k]["group_priority"], rtol=1e-9)
    for f in ("status", "round", "model", "worker", "order"):
        assert np.array_equal(reqs[f], od.reqs[f]), f
    assert np.array_equal(t_w.cpu().numpy(), od.t_end_ns) and np.array_equal(l_w.cpu().numpy(), od.loaded_end)
    if n_workers > 1:
        assert len(np.unique(od.rounds[0, :k]["worker"])) > 1
    ses.close()


def _reference_set(w, r, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal(size=(r, int(w.feat_dim)), dtype=np.float32)
    ref = synth.f32_to_bf16_bits(x) if int(w.feat_dtype) == synth.BF16 else x
    return ref, rng.integers(0, int(w.n_classes), size=r).astype(np.int32), rng.integers(0, int(w.n_apps), size=r).astype(np.int32)


@pytest.mark.parametrize("name,kw,k,prior,mode", [
    ("C1", {}, 5, True, "rounds"), ("C1", {}, 1, False, "split"), ("C2", dict(n_requests=1500, n_classes=12), 17, False, "forced"),
    ("C3", dict(n_requests=800, n_classes=40, feat_dim=128), 5, True, "rounds"), ("C1", dict(n_requests=300), 4000, False, "rounds")])
def test_nearest_neighbour_evidence_matches_oracle(name, kw, k, prior, mode):
    """Section 4.1's SneakPeek model: votes of the k nearest reference points, Dirichlet posterior mean (Eq. 10-11),
    Eq. 9; then the rounds run on those scores (plain, with every decision forced through the fp64 values, or over
    the sub-groups the votes define)."""
    import torch
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload(name, **kw)
    if prior:
        w.prior_alpha = np.full((1, int(w.n_apps), int(w.n_classes)), 0.5, dtype=np.float32)     # Jeffreys
        w.evidence_k = 1.0
    ref, ref_label, ref_app = _reference_set(w, 2000, 5)
    if k > 1000:
        k = 3                                                    # ... and a reference set smaller than k for one application
        keep = (ref_app != 0) | (np.cumsum(ref_app == 0) <= 2)
        ref, ref_label, ref_app = ref[keep], ref_label[keep], ref_app[keep]
    s = oracle.score_knn(w, k, ref, ref_label, ref_app)
    od = oracle.drain(w, s.acc, s.v, labels=s.label if mode == "split" else None)
    n = w.n_requests
    ses = runner.Session(w)
    api.sp_load_evidence(ses.ctx, k, ref, ref_label, ref_app)
    if mode == "forced":
        api.sp_set_options(ses.ctx, trace_mode=False, guard_utility=1.0, guard_priority=1.0)
    ses.upload(); ses.alloc_outputs(n)
    dv = ses.dev
    api.sp_reset(ses.ctx)
    api.sp_set_clocks(ses.ctx, dv["t0"], dv["l0"])
    api.sp_score_knn(ses.ctx, n, dv["feats"], dv["app"], dv["arrival"], dv["deadline"], None)
    if mode == "split":
        api.sp_schedule_split(ses.ctx, ses.rounds, ses.cap, ses.n_done)
    else:
        ses.schedule(n + 1)
    acc = torch.empty((n, ses.mmax), dtype=torch.float32, device=ses.device)
    v = torch.empty(n, dtype=torch.float32, device=ses.device)
    lab = torch.empty(n, dtype=torch.int32, device=ses.device)
    api.sp_get_scores(ses.ctx, 0, n, acc, v)
    api.sp_get_labels(ses.ctx, 0, n, lab)
    api.sp_get_requests(ses.ctx, 0, n, ses.recs)
    t_end = torch.empty(1, dtype=torch.int64, device=ses.device)
    l_end = torch.empty(1, dtype=torch.int32, device=ses.device)
    api.sp_get_clocks(ses.ctx, t_end, l_end)
    api.sp_check(ses.ctx)
    np.testing.assert_allclose(acc.cpu().numpy(), s.acc, rtol=1e-6, atol=1e-30)
    np.testing.assert_allclose(v.cpu().numpy(), s.v, rtol=1e-6)
    assert np.array_equal(lab.cpu().numpy(), s.label)
    res = runner.Result(None, None, ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:n],
                        ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE), ses.n_done.cpu().numpy(),
                        t_end.cpu().numpy(), l_end.cpu().numpy(), api.sp_get_stats(ses.ctx))
    ses.close()
    check_schedule(w, res, od)
    if mode == "forced":
        assert res.stats["exact_utility"] > 0 and res.stats["exact_rows"] == 0     # decided on the neighbour scores, no re-scoring
