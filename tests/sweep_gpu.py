"""Randomized parity sweep of the CUDA library against the CPU oracle (needs a B200; run by hand, not by pytest).

    python tests/sweep_gpu.py SEED N_CASES [--bf16] [--soft] [--short] [--prior] [--resume] [--bmax] [--trace] [--loaded]

Each case draws a seeded shape (applications, models, labels, feature width, requests, instances) around the limits
of the scoring kernels, builds the synthetic workload, and compares scores (1e-5 relative) and the schedule (exact)
with the oracle, as the committed parity tests do.  Options add random penalty kinds, a short-circuit candidate,
Dirichlet priors, rounds run in several calls, other largest batch sizes, trace mode and an initial resident model.
Exit status 1 when a case differs.
"""
import os
import sys
import time
import traceback

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2505_06641_b200 import api, runner, synth          # noqa: E402
from oracle import oracle                                      # noqa: E402
from parity import check_schedule, check_scores                # noqa: E402


def main():
    seed, n_cases = int(sys.argv[1]), int(sys.argv[2])
    opt = set(sys.argv[3:])
    rng = np.random.default_rng(seed)
    bad, t0 = 0, time.time()
    for k in range(n_cases):
        base = "C3" if "--bf16" in opt else ["C4", "C1", "C2", "C5"][k % 4]
        kw = dict(n_apps=int(rng.integers(1, 5)), models=int(rng.integers(1, 9)),
                  n_classes=int(rng.choice([2, 3, 5, 8, 10, 12, 16, 20, 21, 24, 32, 36, 40, 64, 100])),
                  feat_dim=int(rng.choice([32, 64, 96, 128, 160, 256, 512])), n_requests=int(rng.integers(1, 1500)))
        if "--trace" in opt and base in ("C1", "C4") and rng.random() < 0.7:
            kw["trace_mode"] = True
        if "--bmax" in opt:
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
        guards = None if rng.random() < 0.8 else (1.0, 1.0)      # one in five: every decision through the fp64 path
        kinds = rng.integers(0, 3, size=kw["n_apps"]).astype(np.int32) if "--soft" in opt else None
        static_acc = float(rng.uniform(0.3, 0.7)) if "--short" in opt and rng.random() < 0.5 else None
        try:
            w = synth.make_workload(base, **kw)
            if kinds is not None:
                w.penalty_kind = kinds
            if static_acc is not None:
                w = synth.with_short_circuit(w, static_acc)
            if "--prior" in opt and rng.random() < 0.7:
                w.prior_alpha = rng.uniform(0.05, 3.0, size=(int(w.n_instances), int(w.n_apps), int(w.n_classes))).astype(np.float32)
                w.evidence_k = float(rng.uniform(0.5, 20.0))
            s = oracle.score(w)
            od = oracle.drain(w, s.acc, s.v)
            ses = runner.Session(w)
            if guards is not None:
                api.sp_set_options(ses.ctx, trace_mode=bool(w.trace_mode), guard_utility=guards[0], guard_priority=guards[1])
            if "--resume" in opt and int(w.n_instances) == 1:
                step = int(rng.integers(1, 6))
                ses.upload()
                ses.alloc_outputs(64)
                ses.score()
                got = []
                while True:
                    ses.schedule(step)
                    api.sp_check(ses.ctx)
                    done = int(ses.n_done.cpu()[0])
                    got.append(ses.rounds.cpu().numpy().reshape(1, -1).view(api.ROUND_DTYPE)[0, :done].copy())
                    if done < step:
                        break
                got = np.concatenate(got)
                ses.close()
                assert len(got) == od.n_rounds[0], "%d rounds, oracle %d" % (len(got), od.n_rounds[0])
                for f in ("round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"):
                    assert np.array_equal(got[f], od.rounds[0, :len(got)][f]), f
                print("ok  %4d %s %s in calls of %d rounds" % (k, base, kw, step), flush=True)
                continue
            loaded0 = None
            if "--loaded" in opt and rng.random() < 0.6:
                loaded0 = rng.integers(-1, int(np.sum(w.models_per_app)), size=int(w.n_instances)).astype(np.int32)
                od = oracle.drain(w, s.acc, s.v, loaded0=loaded0)
            res = ses.run(loaded0=loaded0)
            ses.close()
            worst = check_scores(res, s)
            skipped = check_schedule(w, res, od)
            print("ok  %4d %s %s kinds=%s static=%s guards=%s worst=%.2e near-ties=%d kernel=%d" % (
                k, base, kw, kinds, static_acc, guards, worst, skipped, res.stats.get("score_kernel", -1)), flush=True)
        except Exception:
            bad += 1
            print("BAD %4d %s %s kinds=%s static=%s guards=%s\n%s" % (k, base, kw, kinds, static_acc, guards,
                                                                      traceback.format_exc()[-800:]), flush=True)
    print("done: %d bad of %d in %.0f s" % (bad, n_cases, time.time() - t0))
    return 1 if bad else 0


if __name__ == "__main__":
    sys.exit(main())
