"""Comparison of the CUDA library's output with the oracle's (test helper)."""
import numpy as np

ACC_RTOL = 1e-5        # data-aware accuracies and utilities, fp32 path vs fp64 oracle
NEAR_TIE = 1e-9        # rounds whose two best utilities / priorities are closer than this are not compared


def check_scores(res, orc, rtol=ACC_RTOL):
    np.testing.assert_allclose(res.acc, orc.acc, rtol=rtol, atol=1e-30)
    np.testing.assert_allclose(res.v, orc.v, rtol=rtol)
    return float(np.max(np.abs(res.acc - orc.acc) / np.maximum(orc.acc, 1e-30)))


def check_schedule(w, res, od):
    """Bit-exact schedule (chosen model, batch membership, order, clock) per instance.

    The oracle reports, per round, the relative gap between its two best group priorities and candidate
    utilities.  From the first round of an instance whose gap is below NEAR_TIE on, that instance is no
    longer compared (either choice is acceptable there); the number of such instances is returned.
    """
    ni = int(w.n_instances)
    inst = np.asarray(w.instance)
    skipped = 0
    int_fields = ["instance", "round", "app", "model", "batch", "n_members", "n_expired", "t_start_ns", "t_end_ns"]
    for k in range(ni):
        nr = int(od.n_rounds[k])
        orr = od.rounds[k, :nr]
        tie = np.nonzero((orr["util_margin"] < NEAR_TIE) | (orr["prio_margin"] < NEAR_TIE))[0]
        upto = int(tie[0]) if len(tie) else nr
        if len(tie):
            skipped += 1
        else:
            assert int(res.n_rounds[k]) == nr, "instance %d: %d rounds, oracle %d" % (k, res.n_rounds[k], nr)
            assert int(res.t_end_ns[k]) == int(od.t_end_ns[k]) and int(res.loaded_end[k]) == int(od.loaded_end[k])
        cap = min(upto, res.rounds.shape[1], od.rounds.shape[1])
        g = res.rounds[k, :cap]
        for f in int_fields:
            bad = np.nonzero(g[f] != orr[f][:cap])[0]
            assert len(bad) == 0, "instance %d round %d: %s = %s, oracle %s" % (
                k, bad[0], f, g[f][bad[0]], orr[f][bad[0]])
        np.testing.assert_allclose(g["utility"], orr["utility"][:cap], rtol=ACC_RTOL)
        np.testing.assert_allclose(g["group_priority"], orr["group_priority"][:cap], rtol=ACC_RTOL)
        sel = np.nonzero(inst == k)[0] if ni > 1 else slice(None)
        o_req, g_req = od.reqs[sel], res.reqs[sel]
        keep = (o_req["round"] >= 0) & (o_req["round"] < upto) if len(tie) else np.ones(len(o_req), dtype=bool)
        for f in ("status", "round", "model", "order"):
            bad = np.nonzero(g_req[f][keep] != o_req[f][keep])[0]
            assert len(bad) == 0, "instance %d request #%d: %s = %s, oracle %s" % (
                k, bad[0], f, g_req[f][keep][bad[0]], o_req[f][keep][bad[0]])
    return skipped
