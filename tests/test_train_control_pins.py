"""Pins for the oracle's Train(student, frame, label) (Algorithm 1): its control flow is checked against
an independent replay — the plain K-step loop, whose parts are pinned elsewhere, with the metric of every
iterate recomputed from scratch and the loop's rules applied to that list by hand.  CPU only."""
import numpy as np
import pytest

import oracle
import synth_inputs as si


def problem(seed=0, c_in=8, c_hidden=0, C=4, h=6, w=9, strength=2.0):
    cls = si.voronoi_map(4 * h, 4 * w, 6, C, 2000 + seed)
    feat = si.label_informed_features(c_in, h, w, cls, 4, seed, strength)
    theta = si.initial_head_params(c_in, c_hidden, C, 1000 + seed)
    return feat, cls, theta


def iterates(feat, labels, theta, c_in, c_hidden, C, lr, mu, n):
    """theta and metric after 0..n plain steps, by the step function and the metric function alone."""
    head = oracle.Head(c_in, c_hidden, C, lr=lr, momentum=mu, theta=theta)
    thetas, metrics = [head.theta.copy()], [oracle.agreement(labels, oracle.student_mask(head, feat), C)[1]]
    for _ in range(n):
        oracle.distill_step(head, feat, labels)
        thetas.append(head.theta.copy())
        metrics.append(oracle.agreement(labels, oracle.student_mask(head, feat), C)[1])
    return thetas, metrics


def by_hand(metrics, threshold, max_updates):
    """Algorithm 1's rules applied to a list of metrics: (n_updates, best_iter)."""
    best, best_i, n = metrics[0], 0, 0
    if metrics[0] < threshold:
        for i in range(1, max_updates + 1):
            n = i
            if metrics[i] > best:
                best, best_i = metrics[i], i
            if metrics[i] > threshold:
                break
    return n, best_i


@pytest.mark.parametrize("c_hidden", [0, 8])
def test_metrics_rise_on_label_informed_features(c_hidden):
    feat, labels, theta = problem(c_hidden=c_hidden)
    _, m = iterates(feat, labels, theta, 8, c_hidden, 4, 0.5, 0.9, 12)
    assert m[-1] > m[0] + 0.2, m          # the workload is learnable, so the rules below have something to decide


def test_threshold_already_met_takes_no_step():
    feat, labels, theta = problem()
    head = oracle.Head(8, 0, 4, lr=0.5, momentum=0.9, theta=theta)
    m0 = oracle.agreement(labels, oracle.student_mask(head, feat), 4)[1]
    for thr in (0.0, m0):                  # "best_metric < THRESHOLD" is false in both cases
        r = oracle.train_key_frame(head, feat, labels, thr, 5)
        assert (r.n_updates, r.best_iter, r.metrics, r.losses) == (0, 0, [m0], [])
        assert r.best_metric == m0
        assert head.theta.tobytes() == np.asarray(theta, np.float32).tobytes()
        assert not head.vel.any()


@pytest.mark.parametrize("c_hidden,mu", [(0, 0.0), (0, 0.9), (8, 0.9)])
def test_unreachable_threshold_runs_all_updates_and_returns_the_best_iterate(c_hidden, mu):
    K = 10
    feat, labels, theta = problem(seed=1, c_hidden=c_hidden)
    thetas, m = iterates(feat, labels, theta, 8, c_hidden, 4, 0.5, mu, K)
    head = oracle.Head(8, c_hidden, 4, lr=0.5, momentum=mu, theta=theta)
    r = oracle.train_key_frame(head, feat, labels, 2.0, K)        # a mean IoU never exceeds 1
    assert r.n_updates == K and r.metrics == m and len(r.losses) == K
    best_i = int(np.argmax(m))                                     # first occurrence of the maximum: "metric > best"
    assert r.best_iter == best_i and r.best_metric == m[best_i] == max(m)
    assert head.theta.tobytes() == thetas[best_i].tobytes()


def test_break_at_first_metric_above_threshold():
    K = 12
    feat, labels, theta = problem(seed=2)
    thetas, m = iterates(feat, labels, theta, 8, 0, 4, 0.5, 0.9, K)
    assert max(m) > m[0]
    seen = set()
    for thr in sorted(set(0.5 * (a + b) for a, b in zip(sorted(m)[:-1], sorted(m)[1:]))) + [m[3], max(m)]:
        n_ref, best_ref = by_hand(m, thr, K)
        head = oracle.Head(8, 0, 4, lr=0.5, momentum=0.9, theta=theta)
        r = oracle.train_key_frame(head, feat, labels, thr, K)
        assert (r.n_updates, r.best_iter) == (n_ref, best_ref), thr
        assert r.metrics == m[:n_ref + 1] and r.best_metric == m[best_ref]
        assert head.theta.tobytes() == thetas[best_ref].tobytes()
        if 0 < n_ref < K:
            assert m[n_ref] > thr and all(x <= thr for x in m[1:n_ref])     # strict ">" ends the loop, not ">="
        seen.add(n_ref)
    assert len(seen) >= 3                  # the thresholds exercised several different exits


def test_a_worse_later_iterate_is_not_returned():
    # a large learning rate makes the metric go up and down; the returned student is the best one seen, not the last
    K = 10
    feat, labels, theta = problem(seed=3)
    thetas, m = iterates(feat, labels, theta, 8, 0, 4, 6.0, 0.9, K)
    best_i = int(np.argmax(m))
    assert best_i != K and m[K] < m[best_i], m     # the case is what it is meant to be
    head = oracle.Head(8, 0, 4, lr=6.0, momentum=0.9, theta=theta)
    r = oracle.train_key_frame(head, feat, labels, 2.0, K)
    assert r.best_iter == best_i and head.theta.tobytes() == thetas[best_i].tobytes()


def test_max_updates_zero():
    feat, labels, theta = problem()
    head = oracle.Head(8, 0, 4, lr=0.5, theta=theta)
    r = oracle.train_key_frame(head, feat, labels, 2.0, 0)
    assert r.n_updates == 0 and len(r.metrics) == 1 and head.theta.tobytes() == np.asarray(theta, np.float32).tobytes()
