"""The allocation-free scoring call, for hosts that may not call cudaMalloc once they are running.

Collected last on purpose (file name): a run that stops at the first failure has then already run every other
test.  The call under test keeps its scratch in a fixed array inside the library, so the things worth checking
are that it gives what the context-based sp_score() gives (and what the CPU oracle gives), that a second call --
which finds the array dirty from the first -- still does, and that the free device memory reported by the driver
is the same after such a call as before it.
"""
import numpy as np
import pytest

from paper_2505_06641_b200 import synth

pytestmark = pytest.mark.gpu


def _reference_scores(w):
    """acc, v from the existing entry point (sp_score + sp_get_scores)."""
    import torch
    from paper_2505_06641_b200 import api, runner
    ses = runner.Session(w)
    ses.upload()
    ses.score()
    acc = torch.empty((ses.n, ses.mmax), dtype=torch.float32, device=ses.device)
    v = torch.empty(ses.n, dtype=torch.float32, device=ses.device)
    api.sp_get_scores(ses.ctx, 0, ses.n, acc, v)
    api.sp_check(ses.ctx)
    out = acc.cpu().numpy(), v.cpu().numpy()
    ses.close()
    return out


def _static_scores(w):
    import torch
    from paper_2505_06641_b200 import api, runner
    dev = torch.device("cuda", 0)
    bf16 = int(w.feat_dtype) == api.SP_BF16
    to = lambda a: runner._bits_tensor(a, dev) if bf16 else torch.from_numpy(a).to(dev)
    head_w, feats = to(w.head_w[0]).contiguous(), to(w.feats).contiguous()
    head_b = torch.from_numpy(w.head_b[0]).to(dev)
    recall = torch.from_numpy(w.recall[0]).to(dev)
    app = torch.from_numpy(np.ascontiguousarray(w.app, dtype=np.int32)).to(dev)
    n, mmax = w.n_requests, w.max_models
    acc = torch.full((n, mmax), -1.0, dtype=torch.float32, device=dev)
    v = torch.full((n,), -1.0, dtype=torch.float32, device=dev)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    api.sp_score_static(0, torch.cuda.current_stream().cuda_stream, w.n_apps, w.n_classes, w.feat_dim, w.feat_dtype,
                        w.models_per_app, head_w, head_b, recall, n, feats, app, acc, v)
    free_after = torch.cuda.mem_get_info(dev)[0]
    return acc.cpu().numpy(), v.cpu().numpy(), free_before - free_after


def test_static_scoring_matches_sp_score_on_two_calls_in_a_row():
    # different shapes back to back: the second call meets counters and a permutation left by the first
    calls = 0
    for name, kw in (("C2", {}), ("C1", {}), ("C3", dict(n_requests=777)), ("C2", dict(n_requests=1000))):
        w = synth.make_workload(name, **kw)
        ref_acc, ref_v = _reference_scores(w)
        acc, v, taken = _static_scores(w)
        np.testing.assert_allclose(acc, ref_acc, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(v, ref_v, rtol=1e-5)
        if calls:                  # (the very first call on a device may load the module that holds the array)
            deltas = [taken] + [_static_scores(w)[2] for _ in range(2 if taken else 0)]
            # the driver's figure is device-wide, so a neighbour may move it once; it must not move with every call
            assert 0 in deltas, "free device memory changed across every call: %s bytes" % deltas
        calls += 1


def test_static_scoring_matches_the_oracle():
    from oracle import oracle
    for name, kw in (("C1", {}), ("C3", dict(n_requests=300))):
        w = synth.make_workload(name, **kw)
        s = oracle.score(w)
        acc, v, _ = _static_scores(w)
        np.testing.assert_allclose(acc, s.acc, rtol=1e-5, atol=1e-30)
        np.testing.assert_allclose(v, s.v, rtol=1e-5)


def test_static_scoring_rejects_what_does_not_fit():
    import torch
    from paper_2505_06641_b200 import api
    w = synth.make_workload("C1")
    dev = torch.device("cuda", 0)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    args = (0, 0, w.n_apps, w.n_classes, w.feat_dim, w.feat_dtype, w.models_per_app, t(w.head_w[0]), t(w.head_b[0]),
            t(w.recall[0]))
    feats, app = t(w.feats), t(w.app.astype(np.int32))
    acc = torch.zeros((w.n_requests, w.max_models), device=dev)
    v = torch.zeros(w.n_requests, device=dev)
    with pytest.raises(api.SpError) as e:
        api.sp_score_static(*args, 65537, feats, app, acc, v)
    assert e.value.status == api.SP_EINVAL and "65536" in str(e.value)
    app[3] = 9                                           # bad application id: reported, outputs untouched
    with pytest.raises(api.SpError) as e:
        api.sp_score_static(*args, w.n_requests, feats, app, acc, v)
    assert e.value.status == api.SP_EINVAL and float(acc.abs().sum()) == 0.0
    app[3] = 0                                           # and the array is usable again afterwards
    api.sp_score_static(*args, w.n_requests, feats, app, acc, v)
    assert float(acc.min()) > 0.0
