"""Pins for the oracle's variant without the exact average (Section 6 of the paper: the outer
update applied by every worker to its own model)."""
import numpy as np
import pytest

import oracle
from test_oracle_pins import N, Problem, close, f32, run64


def test_single_worker_has_nothing_to_average():
    for base in ("nesterov", "adam", "sgp_nesterov"):
        kw = dict(m=1, tau=4, T=4, alpha=0.8, beta=0.5, gamma=0.03, base=base, mu=0.9, sigma=0.2, seed=51,
                  buffer_policy="maintain")
        a = run64(oracle.make_config(no_average=True, **kw))
        b = run64(oracle.make_config(**kw))
        assert np.array_equal(a["anchor"][0], b["anchor"]) and np.array_equal(a["u"][0], b["u"])
        assert np.array_equal(a["x"], b["x"]) and np.array_equal(a["h"], b["h"])


def test_identical_workers_stay_identical_and_match_the_averaged_method():
    # supplied gradients equal on all workers: every worker follows the same path, which is also
    # the path of the averaged method (the mean of equal values is that value, up to rounding)
    m, tau, T, n = 4, 3, 3, 12
    from paper_1910_00643_b200.workloads import dense_gradients
    G = np.repeat(dense_gradients(T * tau, 1, n, seed=8), m, axis=1)
    kw = dict(m=m, tau=tau, T=T, alpha=0.9, beta=0.6, gamma=0.05, mu=0.9, grad_mode="supplied_array",
              buffer_policy="reset")
    a = oracle.run(oracle.make_config(no_average=True, **kw), j0=0, n=n, precision="f64", G=G)
    b = oracle.run(oracle.make_config(**kw), j0=0, n=n, precision="f64", G=G)
    for i in range(m):
        close(a["anchor"][i], b["anchor"], 1e-13)
        close(a["u"][i], b["u"], 1e-12)
        assert np.array_equal(a["anchor"][i], a["anchor"][0])


@pytest.mark.parametrize("base,policy", [("nesterov", "reset"), ("nesterov", "maintain"), ("adam", "maintain")])
def test_without_communication_every_worker_is_its_own_slow_momentum_run(base, policy):
    # communication-free base + no average: worker i never sees the others, so its trajectory is
    # a one-worker slow-momentum (Lookahead with momentum) run on its own data, written here as
    # a textbook loop
    m, tau, T = 3, 4, 5
    kw = dict(m=m, tau=tau, T=T, alpha=0.8, beta=0.5, gamma=0.01 if base == "adam" else 0.06, base=base, mu=0.9,
              sigma=0.2, weight_decay=1e-3, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-7, buffer_policy=policy, seed=52,
              x_init=0.2)
    cfg = oracle.make_config(no_average=True, **kw)
    p = Problem(cfg)
    out = run64(cfg)
    gam, alpha, beta = f32(kw["gamma"]), f32(0.8), f32(0.5)
    mu, b1, b2, eps = f32(0.9), f32(0.9), f32(0.98), f32(1e-7)
    for i in range(m):
        slow = np.full(N, f32(0.2)); u = np.zeros(N); h = np.zeros(N); v = np.zeros(N); l = 0
        for t in range(T):
            fast = slow.copy()
            for k in range(tau):
                g = p.grad(t, k, i, fast)
                if base == "adam":
                    l += 1
                    h = b1 * h + (1 - b1) * g
                    v = b2 * v + (1 - b2) * g * g
                    d = (h / (1 - b1 ** l)) / (np.sqrt(v / (1 - b2 ** l)) + eps)
                else:
                    h = mu * h + g
                    d = mu * h + g
                fast = fast - gam * d
            u = beta * u + (slow - fast) / gam
            slow = slow - alpha * gam * u
            if policy == "reset":
                h = np.zeros(N); v = np.zeros(N); l = 0
        close(out["anchor"][i], slow, 1e-11)
        close(out["u"][i], u, 1e-10)
        close(out["x"][i], slow, 1e-11)
        close(out["h"][i], h, 1e-11)


def test_worker_means_obey_the_outer_update_with_sgp_base():
    # the outer update is linear, so the worker means satisfy Eq. (2), (3) with the mean model;
    # push-sum mixing keeps the mean step equal to -gamma * (mean direction)
    kw = dict(m=4, tau=5, alpha=1.0, beta=0.6, gamma=0.04, base="sgp_nesterov", mu=0.9, sigma=0.3, seed=53,
              buffer_policy="maintain", no_average=True)
    T = 4
    xs, us = [np.zeros(N)], [np.zeros(N)]
    for t in range(1, T + 1):
        last = run64(oracle.make_config(T=t, **kw), want_dbar=True)
        xs.append(last["anchor"].mean(axis=0)); us.append(last["u"].mean(axis=0))
    D = last["dbar"].sum(axis=1)
    gam, beta = f32(0.04), f32(0.6)
    for t in range(T):
        close(us[t + 1], beta * us[t] + D[t], 1e-10)
        close(xs[t + 1], xs[t] - gam * us[t + 1], 1e-11)
    # without the average the workers do not agree after the outer step
    assert np.abs(last["anchor"] - last["anchor"][0]).max() > 1e-4


def test_average_policy_is_rejected_without_the_average():
    with pytest.raises(ValueError):
        oracle.run(oracle.make_config(m=2, tau=1, T=1, no_average=True, buffer_policy="average"), j0=0, n=1)
