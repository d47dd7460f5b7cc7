"""Parity with the CPU oracle at the full size of the large configurations, and on the kernel paths that only
large inputs reach (several tiles per block in the GEMM-shaped scoring kernels).  Needs a B200; run with -m gpu.

The oracle scores every request of these workloads in fp64 on the host cores (a few seconds to a minute each),
so the comparison is element by element over the whole table, not a sample.
"""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth
from parity import ACC_RTOL, check_schedule, check_scores

pytestmark = pytest.mark.gpu


def _both(w, **kw):
    from oracle import oracle
    from paper_2505_06641_b200 import runner
    s = oracle.score(w)
    od = oracle.drain(w, s.acc, s.v)
    ses = runner.Session(w)
    res = ses.run(**kw)
    ses.close()
    return s, od, res


def _tiles_per_block(w, rows_per_tile=128, n_blocks=148):
    groups = np.bincount(np.asarray(w.instance).astype(np.int64) * int(w.n_apps) + np.asarray(w.app),
                         minlength=int(w.n_instances) * int(w.n_apps))
    return int(np.sum((groups + rows_per_tile - 1) // rows_per_tile)) / n_blocks


def test_bf16_head_with_several_tiles_per_block_and_two_label_chunks():
    """25,000 requests x 256 features x 512 labels in bf16: 197 tiles of 128 requests on 148 blocks, two chunks of
    256 logit columns per tile, so blocks wrap their operand rings and reuse both accumulators across tiles."""
    w = synth.make_workload("C3", n_requests=25000, n_classes=512, feat_dim=256)
    assert _tiles_per_block(w) > 1.0
    s, od, res = _both(w)
    assert res.stats["score_kernel"] == 3
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)


def test_fp32_gemm_head_with_several_tiles_per_block():
    """The tf32-split flavour of the same kernel on 40,000 requests x 256 features x 200 labels (313 tiles)."""
    w = synth.make_workload("C5", n_requests=40000, feat_dim=256)
    assert _tiles_per_block(w) > 2.0
    s, od, res = _both(w)
    assert res.stats["score_kernel"] == 4
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)


def test_large_class_configuration_at_full_size():
    """C3 as specified: 65,536 requests x 1,024 bf16 features x 1,000 labels, 3 x 16 models (512 tiles on 148 blocks,
    four label chunks); every accuracy, every variance factor and the whole schedule against the oracle."""
    w = synth.make_workload("C3")
    assert w.n_requests == 65536 and w.n_classes == 1000 and w.feat_dim == 1024
    s, od, res = _both(w)
    assert res.stats["score_kernel"] == 3
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)
    assert np.all(res.reqs["status"] != 0)


def test_trace_replay_configuration_at_full_size():
    """C5 as specified: 1,000,000 requests in trace mode (about 18,000 rounds back to back on the device with arrivals
    joining between rounds); scores and the whole schedule against the oracle."""
    w = synth.make_workload("C5")
    assert w.n_requests == 1_000_000 and w.trace_mode
    s, od, res = _both(w)
    assert res.stats["score_kernel"] == 4
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)
    assert np.all(res.reqs["status"] != 0)


def _with_prior(w, seed):
    rng = np.random.default_rng(seed)
    w.prior_alpha = rng.uniform(0.05, 3.0, size=(int(w.n_instances), int(w.n_apps), int(w.n_classes))).astype(np.float32)
    w.evidence_k = float(rng.uniform(2.0, 20.0))
    return w


@pytest.mark.parametrize("name,kw,kernel", [
    ("C1", {}, 2),                                              # tensor-core small-head kernel, one instance
    ("C4", dict(n_instances=300), 2),                           # ... many instances per block
    ("C3", dict(n_requests=20000, n_classes=512, feat_dim=256), 3),   # bf16 GEMM-shaped kernel, several tiles per block
    ("C2", dict(n_requests=20000), 4),                          # fp32 GEMM-shaped kernel
    ("C2", dict(n_requests=500, n_classes=30, feat_dim=200), 1),      # FP32-ALU small-head kernel
    ("C2", dict(n_requests=500, n_classes=101), 0)])            # FP32-ALU tiled kernel
def test_dirichlet_prior_on_every_scoring_kernel(name, kw, kernel):
    """Eq. 10-11 with a random prior and evidence weight, on each of the scoring kernels."""
    w = _with_prior(synth.make_workload(name, **kw), 77)
    s, od, res = _both(w)
    assert res.stats["score_kernel"] == kernel
    assert check_scores(res, s) < ACC_RTOL
    check_schedule(w, res, od)
    # the prior really changed the scores
    w0 = synth.make_workload(name, **kw)
    from oracle import oracle
    assert np.max(np.abs(oracle.score(w0).acc - s.acc)) > 1e-3
