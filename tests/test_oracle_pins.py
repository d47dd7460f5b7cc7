"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed)."""
import os

import numpy as np
import pytest
from scipy.special import softmax

from oracle import oracle
from paper_2505_06641_b200 import synth
from helpers import (MS, brute_force_request_level, first_model, manual_workload, replay_schedule)

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    rows = [l.split() for l in open(os.path.join(GOLD, name)) if l.strip() and not l.startswith("#")]
    return np.asarray(rows, dtype=np.float64)


def _simple(acc_probs, recall, **kw):
    n = len(acc_probs)
    m = len(recall)
    args = dict(app=[0] * n, deadline_ms=[1e6] * n, alpha_ms=[1.0] * m, beta_ms=[1.0] * m,
                swap_ms=[0.0] * m, batch_sizes=[1], models_per_app=[m])
    args.update(kw)
    return manual_workload(acc_probs, recall, **args)


# ------------------------------------------------------------------ scoring (a1-a4)

def test_dirichlet_worked_example():
    """Section 4.1: y = <2,3>, Jeffreys prior 0.5 => posterior mean (2.5/6, 3.5/6)."""
    a1, a2, y1, y2, m1, m2 = _gold("dirichlet_fall_example.txt")[0]
    k = y1 + y2
    w = _simple([[y1 / k, y2 / k]], [[1.0, 0.0], [0.0, 1.0]], prior_alpha=[[a1, a2]], evidence_k=k)
    s = oracle.score(w, want_theta=True)
    np.testing.assert_allclose(s.theta[0], [m1, m2], rtol=0, atol=2e-7)
    # recall = identity rows => accuracy of "model c" is theta_c itself
    np.testing.assert_allclose(s.acc[0], [m1, m2], rtol=0, atol=2e-7)


def test_dirichlet_limits():
    p = [[0.2, 0.3, 0.5]]
    rec = [[0.9, 0.5, 0.1]]
    no_prior = oracle.score(_simple(p, rec), want_theta=True).theta[0]
    np.testing.assert_allclose(no_prior, p[0], atol=2e-7)
    zero_prior = oracle.score(_simple(p, rec, prior_alpha=[[0, 0, 0]], evidence_k=3.0), want_theta=True).theta[0]
    np.testing.assert_allclose(zero_prior, p[0], atol=2e-7)
    huge = oracle.score(_simple(p, rec, prior_alpha=[[6e6, 3e6, 1e6]], evidence_k=1.0), want_theta=True).theta[0]
    np.testing.assert_allclose(huge, [0.6, 0.3, 0.1], atol=1e-6)


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", dict(n_requests=300)), ("C3", dict(n_requests=64)),
                                     ("C4", dict(n_instances=3))])
def test_softmax_and_contraction_against_scipy(name, kw):
    """Library second opinion: scipy softmax + einsum in fp64 on the same bytes."""
    w = synth.make_workload(name, **kw)
    s = oracle.score(w, want_theta=True)
    x = synth.bf16_bits_to_f32(w.feats) if w.feat_dtype == synth.BF16 else w.feats
    hw = synth.bf16_bits_to_f32(w.head_w) if w.feat_dtype == synth.BF16 else w.head_w
    x, hw = x.astype(np.float64), hw.astype(np.float64)
    m = w.max_models
    for i in range(0, w.n_requests, 7):
        k, a = int(w.instance[i]), int(w.app[i])
        z = x[i] @ hw[k, a] + w.head_b[k, a].astype(np.float64)
        th = softmax(z)
        np.testing.assert_allclose(s.theta[i], th, rtol=1e-11, atol=1e-300)
        r = w.recall[k, first_model(w, a):first_model(w, a) + m].astype(np.float64)
        acc = np.einsum("c,jc->j", th, r)
        np.testing.assert_allclose(s.acc[i, :m], acc, rtol=1e-11)
        np.testing.assert_allclose(s.v[i], 1.0 + np.var(acc), rtol=1e-12)
    np.testing.assert_allclose(s.theta.sum(axis=1), 1.0, rtol=1e-12)


def test_softmax_shift_invariance():
    w = synth.make_workload("C1")
    a = oracle.score(w, want_theta=True).theta
    w.head_b = w.head_b + np.float32(3.0)          # same shift on every class of every head
    b = oracle.score(w, want_theta=True).theta
    np.testing.assert_allclose(a, b, rtol=1e-6)


def test_eq7_equals_eq9_on_confusion_matrices():
    """tr(Z)/sum(Z) (Eq. 7) equals sum_c theta_c recall_c (Eq. 9) when theta = test-set class frequencies."""
    rng = np.random.default_rng(7)
    for c in (2, 6, 7, 11):
        zs = rng.integers(1, 60, size=(3, c, c)).astype(np.float64)      # three models
        zs[1:] *= zs[0].sum(axis=1, keepdims=True) / zs[1:].sum(axis=2, keepdims=True)  # same test set => same row sums
        theta = zs[0].sum(axis=1) / zs[0].sum()
        recall = np.stack([np.diag(z) / z.sum(axis=1) for z in zs])
        s = oracle.score(_simple([theta], recall))
        eq7 = np.asarray([np.trace(z) / z.sum() for z in zs])
        np.testing.assert_allclose(s.acc[0], eq7, rtol=3e-7)              # fp32 storage of log(theta), recall


def test_one_hot_and_uniform_special_cases():
    rec = np.asarray([[0.9, 0.2, 0.55], [0.1, 0.8, 0.65]])
    eye = np.eye(3)
    s = oracle.score(_simple(eye, rec))
    np.testing.assert_allclose(s.acc, rec.T.astype(np.float32), rtol=1e-12)   # "true model accuracy" of Section 5.3.1
    s = oracle.score(_simple([[0.2, 0.5, 0.3]], np.full((2, 3), 0.75)))
    np.testing.assert_allclose(s.acc[0], [0.75, 0.75], rtol=1e-7)
    assert abs(s.v[0] - 1.0) < 1e-13


def test_priority_factor_hand_worked():
    a1, a2, v = _gold("priority_two_models.txt")[0]
    s = oracle.score(_simple([[1.0, 0.0]], [[a1, 0.3], [a2, 0.3]]))
    np.testing.assert_allclose(s.acc[0], [np.float32(a1), np.float32(a2)], rtol=1e-12)
    assert abs(s.v[0] - v) < 1e-7
    single = oracle.score(_simple([[0.3, 0.7]], [[0.4, 0.9]]))
    assert single.v[0] == 1.0                                                 # footnote of Eq. 12


def test_ragged_models_per_app_pad_with_zero():
    w = manual_workload([[0.5, 0.5]] * 2, [[0.8, 0.6], [0.4, 0.2], [0.9, 0.7]], app=[0, 1], deadline_ms=[1e6] * 2,
                        alpha_ms=[1] * 3, beta_ms=[1] * 3, swap_ms=[0] * 3, batch_sizes=[1], models_per_app=[1, 2])
    s = oracle.score(w)
    np.testing.assert_allclose(s.acc, [[0.7, 0.0], [0.3, 0.8]], rtol=1e-6)
    assert s.v[0] == 1.0 and abs(s.v[1] - (1 + 0.0625)) < 1e-6


# ------------------------------------------------------------------ penalties of Section 5.1 (read as a penalty that grows over the relative deadline)
@pytest.mark.parametrize("kind", [1, 2])
def test_soft_penalties_anchor_points_and_monotonicity(kind):
    """gamma is 0 up to the deadline, 1/2 when late by half the relative deadline, 1 from a whole relative deadline
    on, and never decreases with the completion time (the garbled print fixes no more than that)."""
    from oracle import oracle
    arrival, d = 1_000_000, 5_000_000                     # relative deadline 4 ms
    delta = d - arrival
    assert oracle.penalty(kind, d, arrival, d - 1) == 0.0 and oracle.penalty(kind, d, arrival, d) == 0.0
    assert oracle.penalty(kind, d, arrival, d + delta // 2) == pytest.approx(0.5, abs=1e-15)
    assert oracle.penalty(kind, d, arrival, d + delta) == 1.0 and oracle.penalty(kind, d, arrival, d + 10 * delta) == 1.0
    g = [oracle.penalty(kind, d, arrival, d + k * delta // 1000) for k in range(0, 1001)]
    assert all(b >= a for a, b in zip(g, g[1:])) and g[0] == 0.0 and g[-1] == 1.0
    if kind == 1:
        assert g[250] == pytest.approx(0.25, abs=1e-15)
    else:                                                 # the sigmoid is symmetric about the half-way point
        assert g[250] + g[750] == pytest.approx(1.0, abs=1e-15) and g[250] < 0.25


def test_sigmoid_penalty_rounds_to_one_in_fp64_just_before_the_whole_relative_deadline():
    """1 / (1 + ((1 - x) / x)^3) rounds to 1.0 once ((1 - x) / x)^3 drops below half an ulp of 1, i.e. from
    x = 1 - 4.8e-6 on; the linear penalty stays below 1 until x = 1.  Hopeless is x >= 1 on the integer times, so a
    sigmoid request that is late by all but a few millionths of its relative deadline stays in its queue and, served
    then, earns exactly nothing; one that is late by the whole relative deadline is retired."""
    from oracle import oracle
    from helpers import manual_workload
    arrival, d = 0, 1_000_000_000                         # relative deadline 1 s
    for late_ns, expect_one in ((999_990_000, False), (999_996_000, True), (999_999_999, True)):
        g = oracle.penalty(2, d, arrival, d + late_ns)
        assert (g == 1.0) == expect_one and g <= 1.0
        assert oracle.penalty(1, d, arrival, d + late_ns) < 1.0
    # request 0: deadline 0.9 s, request 1: deadline 1 s; the only candidate completes 1.999996 s after the arrivals
    w = manual_workload([[0.5, 0.5]] * 2, [[0.8, 0.8]], app=[0, 0], deadline_ms=[900, 1000], alpha_ms=[1], beta_ms=[1],
                        swap_ms=[0], batch_sizes=[1], models_per_app=[1], t0_ms=1997.996)
    w.penalty_kind[:] = 2
    s = oracle.score(w)
    dr = oracle.drain(w, s.acc, s.v)
    assert list(dr.reqs["status"]) == [oracle.EXPIRED, oracle.SCHEDULED]
    assert dr.n_rounds[0] == 1 and dr.rounds[0, 0]["utility"] == 0.0 and dr.rounds[0, 0]["n_expired"] == 1


def test_step_penalty_and_degenerate_relative_deadline():
    from oracle import oracle
    assert oracle.penalty(0, 10, 0, 10) == 0.0 and oracle.penalty(0, 10, 0, 11) == 1.0
    for kind in (1, 2):                                   # deadline not after arrival: nothing to scale by
        assert oracle.penalty(kind, 10, 10, 10) == 0.0 and oracle.penalty(kind, 10, 12, 11) == 1.0
