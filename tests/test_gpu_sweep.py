"""A bounded, seeded slice of a randomized parity sweep: 60 shapes around the limits of the scoring kernels with every
option drawn at random (penalty kinds, short-circuit candidate, Dirichlet prior, largest batch size, trace mode, an
initial resident model, all decisions forced through the fp64 path, rounds run in several calls).  Each case is
compared with the CPU oracle like the other parity tests: scores within 1e-5 relative, schedule exact.
Needs a B200; run with -m gpu.
"""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth
from parity import ACC_RTOL, check_schedule, check_scores

pytestmark = pytest.mark.gpu

N_CASES = 60


def _draw_case(k):
    rng = np.random.default_rng(9000 + k)
    base = ["C4", "C1", "C2", "C5", "C3"][k % 5]
    kw = dict(n_apps=int(rng.integers(1, 5)), models=int(rng.integers(1, 9)),
              n_classes=int(rng.choice([2, 3, 5, 8, 10, 12, 16, 20, 21, 24, 32, 36, 40, 64, 100])),
              feat_dim=int(rng.choice([32, 64, 96, 128, 160, 256, 512])), n_requests=int(rng.integers(1, 1500)))
    if base in ("C1", "C4") and rng.random() < 0.5:
        kw["trace_mode"] = True
    if rng.random() < 0.5:
        kw["bmax"] = int(rng.choice([1, 2, 8, 32, 128, 256]))
    if base == "C4":
        kw["n_instances"] = int(rng.choice([2, 37, 400, 1500]))
        kw["n_requests"] = int(rng.integers(1, 400))
    if base == "C3":
        kw["feat_dim"] = int(rng.choice([64, 128, 256, 512, 1024]))
        kw["n_requests"] = int(rng.integers(1, 2500))
        kw["n_classes"] = int(rng.choice([8, 20, 32, 64, 100, 256, 500, 1000]))
    if base == "C5":
        kw["n_requests"] = int(rng.integers(1, 6000))
    opts = dict(
        guards=(1.0, 1.0) if rng.random() < 0.2 else None,
        kinds=rng.integers(0, 3, size=kw["n_apps"]).astype(np.int32) if rng.random() < 0.5 else None,
        static_acc=float(rng.uniform(0.3, 0.7)) if rng.random() < 0.3 else None,
        prior=rng.random() < 0.4, resume=int(rng.integers(1, 6)) if rng.random() < 0.25 else 0,
        loaded=rng.random() < 0.4, seed=int(rng.integers(1 << 30)))
    return base, kw, opts


@pytest.mark.parametrize("k", range(N_CASES))
def test_random_shape_with_random_options(k):
    from oracle import oracle
    from paper_2505_06641_b200 import api, runner
    base, kw, o = _draw_case(k)
    rng = np.random.default_rng(o["seed"])
    w = synth.make_workload(base, **kw)
    if o["kinds"] is not None:
        w.penalty_kind = o["kinds"]
    if o["static_acc"] is not None:
        w = synth.with_short_circuit(w, o["static_acc"])
    if o["prior"]:
        w.prior_alpha = rng.uniform(0.05, 3.0, size=(int(w.n_instances), int(w.n_apps), int(w.n_classes))).astype(np.float32)
        w.evidence_k = float(rng.uniform(0.5, 20.0))
    loaded0 = None
    if o["loaded"]:
        loaded0 = rng.integers(-1, int(np.sum(w.models_per_app)), size=int(w.n_instances)).astype(np.int32)
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v, loaded0=loaded0)
    ses = runner.Session(w)
    if o["guards"] is not None:
        api.sp_set_options(ses.ctx, trace_mode=bool(w.trace_mode), guard_utility=1.0, guard_priority=1.0)
    if o["resume"] and int(w.n_instances) == 1 and loaded0 is None:
        step = o["resume"]
        ses.upload(); ses.alloc_outputs(64); ses.score()
        got = []
        for _ in range(w.n_requests + 2):
            ses.schedule(step)
            api.sp_check(ses.ctx)
            done = int(ses.n_done.cpu()[0])
            got.append(ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE)[0, :done].copy())
            if done < step:
                break
        got = np.concatenate(got)
        ses.close()
        assert len(got) == od.n_rounds[0]
        for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
            assert np.array_equal(got[f], od.rounds[0, :len(got)][f]), f
        return
    res = ses.run(loaded0=loaded0)
    ses.close()
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)
