"""Requests appended to a scored table (a second, third ... sp_score call without sp_reset): the scheduler of a live
system scores what arrived during the last window and goes on with its rounds.  Needs a B200; run with -m gpu."""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth
from parity import ACC_RTOL, check_schedule, check_scores

pytestmark = pytest.mark.gpu


def _score_part(ses, lo, hi):
    from paper_2505_06641_b200 import api
    dv = ses.dev
    api.sp_score(ses.ctx, hi - lo, dv["feats"][lo:hi], dv["app"][lo:hi], dv["arrival"][lo:hi], dv["deadline"][lo:hi], None, None)


def _collect(ses, w):
    import torch
    from paper_2505_06641_b200 import api, runner
    n = ses.n
    acc = torch.empty((n, ses.mmax), dtype=torch.float32, device=ses.device)
    v = torch.empty(n, dtype=torch.float32, device=ses.device)
    api.sp_get_scores(ses.ctx, 0, n, acc, v)
    api.sp_get_requests(ses.ctx, 0, n, ses.recs)
    t_end = torch.empty(1, dtype=torch.int64, device=ses.device)
    l_end = torch.empty(1, dtype=torch.int32, device=ses.device)
    api.sp_get_clocks(ses.ctx, t_end, l_end)
    api.sp_check(ses.ctx)
    return runner.Result(acc.cpu().numpy(), v.cpu().numpy(), ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:n],
                         ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE), ses.n_done.cpu().numpy(),
                         t_end.cpu().numpy(), l_end.cpu().numpy(), api.sp_get_stats(ses.ctx))


@pytest.mark.parametrize("name,kw", [
    ("C1", {}),                                                   # tensor-core small-head kernel
    ("C2", {}),                                                   # fp32 GEMM-shaped kernel
    ("C3", dict(n_requests=3000)),                                # bf16 GEMM-shaped kernel
    ("C2", dict(n_requests=900, n_classes=30, feat_dim=200)),     # FP32-ALU small-head kernel
    ("C2", dict(n_requests=900, n_classes=101)),                  # FP32-ALU tiled kernel
    ("C2", dict(n_requests=20000))])                              # more requests than one block sorts in shared memory
def test_three_calls_give_the_table_of_one_call(name, kw):
    """The requests of a snapshot scored in three calls: same scores, and the rounds that follow are the oracle's."""
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload(name, **kw)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    n = w.n_requests
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(max(1, min(n, 4096)))
    api.sp_reset(ses.ctx)
    api.sp_set_clocks(ses.ctx, ses.dev["t0"], ses.dev["l0"])
    cuts = [0, (n // 3) & ~7, (2 * n // 3 + 5) & ~7, n]
    for lo, hi in zip(cuts, cuts[1:]):
        _score_part(ses, lo, hi)
    ses.schedule(n + 1)
    res = _collect(ses, w)
    ses.close()
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)


@pytest.mark.parametrize("name,kw,kinds", [("C5", dict(n_requests=6000), None), ("C1", dict(n_requests=700, trace_mode=True), [2, 0, 1])])
def test_live_loop_of_rounds_and_appends_equals_the_trace_replay(name, kw, kinds):
    """Trace mode, the way a serving loop uses the library: two rounds, then the requests that arrived meanwhile are
    scored and appended, two more rounds, ...  The schedule must be the one the oracle gives when it knows the whole
    trace in advance."""
    import torch
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload(name, **kw)
    if kinds is not None:
        w.penalty_kind = np.asarray(kinds, dtype=np.int32)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    n, arr = w.n_requests, np.asarray(w.arrival_ns)
    bmax = int(w.batch_sizes[-1])
    horizon = 2 * int(w.swap_ns.max() + w.lat_alpha_ns.max() + w.lat_beta_ns.max() * bmax)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(2)
    api.sp_reset(ses.ctx)
    api.sp_set_clocks(ses.ctx, ses.dev["t0"], ses.dev["l0"])
    t_dev = torch.empty(1, dtype=torch.int64, device=ses.device)
    pos, clock, got, calls = 0, int(w.t0_ns[0]), [], 0
    while True:
        base = max(clock, int(arr[min(pos, n - 1)]))
        upto = max(int(np.searchsorted(arr, base + horizon, side="right")), min(pos + 1, n))
        if upto > pos:
            _score_part(ses, pos, upto)
            pos = upto
        ses.schedule(2)
        api.sp_get_clocks(ses.ctx, t_dev, None)
        api.sp_check(ses.ctx)
        k = int(ses.n_done.cpu()[0])
        got.append(ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE)[0, :k].copy())
        clock = int(t_dev.cpu()[0])
        calls += 1
        if k < 2 and pos == n:
            break
        assert calls < 4 * n
    got = np.concatenate(got)
    assert calls > 10 and len(got) == od.n_rounds[0]
    for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
        assert np.array_equal(got[f], od.rounds[0, :len(got)][f]), f
    np.testing.assert_allclose(got["utility"], od.rounds[0, :len(got)]["utility"], rtol=ACC_RTOL)
    api.sp_get_requests(ses.ctx, 0, n, ses.recs)
    reqs = ses.recs.cpu().numpy().reshape(-1).view(api.REQ_DTYPE)[:n]
    for f in ("status", "round", "model", "order"):
        assert np.array_equal(reqs[f], od.reqs[f]), f
    ses.close()


def test_appended_rows_keep_the_fp64_path_working():
    """With guards of 1.0 every decision re-scores rows in fp64 from the raw features, which after an append live in
    several caller arrays."""
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C2", n_requests=1200)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    n = w.n_requests
    ses = runner.Session(w)
    api.sp_set_options(ses.ctx, trace_mode=False, guard_utility=1.0, guard_priority=1.0)
    ses.upload(); ses.alloc_outputs(n)
    api.sp_reset(ses.ctx)
    api.sp_set_clocks(ses.ctx, ses.dev["t0"], ses.dev["l0"])
    for lo, hi in ((0, 400), (400, 1000), (1000, n)):
        _score_part(ses, lo, hi)
    ses.schedule(n + 1)
    res = _collect(ses, w)
    ses.close()
    assert res.stats["exact_rows"] > 0
    check_schedule(w, res, od)


def test_append_is_refused_where_it_is_not_supported():
    from paper_2505_06641_b200 import api, runner
    w = synth.make_workload("C4", n_instances=3)
    ses = runner.Session(w)
    ses.upload(); ses.alloc_outputs(4); ses.score()
    dv = ses.dev
    with pytest.raises(api.SpError) as e:
        api.sp_score(ses.ctx, 8, dv["feats"][:8], dv["app"][:8], dv["arrival"][:8], dv["deadline"][:8], dv["instance"][:8], None)
    assert e.value.status == api.SP_ESTATE
    ses.close()
    w = synth.make_workload("C1", trace_mode=True)                 # trace mode: an appended request may not arrive
    ses = runner.Session(w)                                        # before the last one already in the table
    ses.upload(); ses.alloc_outputs(4)
    api.sp_reset(ses.ctx)
    _score_part(ses, 100, 200)
    _score_part(ses, 0, 50)
    with pytest.raises(api.SpError) as e:
        api.sp_check(ses.ctx)
    assert e.value.status == api.SP_EINVAL
    ses.close()
