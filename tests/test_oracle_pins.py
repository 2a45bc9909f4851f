"""Pins for the oracle's Algorithm 1: the special cases, identities and closed forms that the
paper's statements fix, library optimizers, and an independently structured brute force.

Each reference below is written from the textbook form of the method it names, not from
the oracle's loop; gradients are rebuilt from the (separately pinned) noise stream.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle

N = 24  # coordinates per case


class Problem:
    """The synthetic quadratic as data: a[j], c[i,j] and noise z[t,k,i,j] in float64."""

    def __init__(self, cfg, n=N):
        self.cfg = cfg
        j = np.arange(n)
        self.a = oracle.curvature(cfg, j).astype(np.float64)
        self.c = np.stack([oracle.centre(cfg, i, j) for i in range(cfg.m)]).astype(np.float64)
        self.sigma = float(np.float32(cfg.sigma))
        self.wd = float(np.float32(cfg.weight_decay))
        self.n = n

    def z(self, t, k, i):
        _, z = oracle.stream(oracle.TAG_GRADNOISE, self.cfg.seed, t, k, i, 0, self.n, words=False)
        return z.astype(np.float64)

    def grad(self, t, k, i, x):
        return self.a * (x - self.c[i]) + self.sigma * self.z(t, k, i) + self.wd * x


def f32(v):
    return float(np.float32(v))


def run64(cfg, **kw):
    return oracle.run(cfg, j0=0, n=N, precision="f64", **kw)


def close(a, b, tol=1e-12):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    assert np.abs(a - b).max() <= tol * (1.0 + np.abs(b).max()), np.abs(a - b).max()


# ---------------------------------------------------------------- special cases of Section 2

def test_tau1_alpha1_is_large_minibatch_heavy_ball_sgd():
    # base SGD, tau = 1, alpha = 1, beta in [0,1): minibatch SGD with momentum beta, lr gamma
    cfg = oracle.make_config(m=5, tau=1, T=9, alpha=1.0, beta=0.8, gamma=0.07, mu=0.0, sigma=0.3, seed=3)
    p = Problem(cfg)
    gam, beta = f32(0.07), f32(0.8)
    x = np.zeros(N)
    vel = np.zeros(N)
    for t in range(9):
        gbar = np.mean([p.grad(t, 0, i, x) for i in range(5)], axis=0)
        vel = beta * vel + gbar
        x = x - gam * vel
    out = run64(cfg)
    close(out["anchor"], x)
    close(out["u"], vel)


def test_beta0_alpha1_is_local_sgd():
    # base SGD, tau > 1, alpha = 1, beta = 0: workers run alone, then x <- average
    cfg = oracle.make_config(m=4, tau=6, T=5, alpha=1.0, beta=0.0, gamma=0.05, mu=0.0, sigma=0.2, seed=1)
    p = Problem(cfg)
    gam = f32(0.05)
    xs = [np.zeros(N) for _ in range(4)]
    for t in range(5):
        for k in range(6):
            xs = [xs[i] - gam * p.grad(t, k, i, xs[i]) for i in range(4)]
        avg = sum(xs) / 4.0
        xs = [avg.copy() for _ in range(4)]
    out = run64(cfg)
    close(out["anchor"], xs[0])
    for i in range(4):
        close(out["x"][i], xs[0])


def test_tau1_beta0_averaged_buffers_is_synchronous_nesterov_sgd():
    # tau = 1, alpha = 1, beta = 0, buffers averaged: one shared Nesterov buffer driven by
    # the mean gradient (fully synchronous SGD)
    cfg = oracle.make_config(m=6, tau=1, T=12, alpha=1.0, beta=0.0, gamma=0.05, mu=0.9, sigma=0.1,
                             weight_decay=1e-3, buffer_policy="average", seed=2)
    p = Problem(cfg)
    gam, mu = f32(0.05), f32(0.9)
    x = np.zeros(N)
    h = np.zeros(N)
    for t in range(12):
        gbar = np.mean([p.grad(t, 0, i, x) for i in range(6)], axis=0)
        h = mu * h + gbar
        x = x - gam * (mu * h + gbar)
    out = run64(cfg)
    close(out["anchor"], x)
    for i in range(6):
        close(out["h"][i], h)


def test_single_worker_beta0_is_lookahead():
    # m = 1, beta = 0, alpha in (0,1]: slow weights move a fraction alpha towards the fast ones
    cfg = oracle.make_config(m=1, tau=5, T=7, alpha=0.5, beta=0.0, gamma=0.1, mu=0.0, sigma=0.2, seed=5)
    p = Problem(cfg)
    gam, alpha = f32(0.1), 0.5
    slow = np.zeros(N)
    for t in range(7):
        fast = slow.copy()
        for k in range(5):
            fast = fast - gam * p.grad(t, k, 0, fast)
        slow = slow + alpha * (fast - slow)
    close(run64(cfg)["anchor"], slow)


@pytest.mark.parametrize("policy", ["maintain", "average"])
def test_local_nesterov_and_double_averaging(policy):
    # Algorithms 4 and 5 of the appendix: per-worker Nesterov buffers, parameters averaged
    # every tau steps; Algorithm 5 also averages the buffers
    cfg = oracle.make_config(m=3, tau=4, T=6, alpha=1.0, beta=0.0, gamma=0.05, mu=0.9, sigma=0.1,
                             buffer_policy=policy, seed=6)
    p = Problem(cfg)
    gam, mu = f32(0.05), f32(0.9)
    xs = [np.zeros(N) for _ in range(3)]
    hs = [np.zeros(N) for _ in range(3)]
    for t in range(6):
        for k in range(4):
            for i in range(3):
                g = p.grad(t, k, i, xs[i])
                hs[i] = mu * hs[i] + g
                xs[i] = xs[i] - gam * (mu * hs[i] + g)
        avg = sum(xs) / 3.0
        xs = [avg.copy() for _ in range(3)]
        if policy == "average":
            havg = sum(hs) / 3.0
            hs = [havg.copy() for _ in range(3)]
    out = run64(cfg)
    close(out["anchor"], xs[0])
    for i in range(3):
        close(out["h"][i], hs[i])


# ------------------------------------------------- identities of the "Equivalent Updates" section

def _anchors(cfg_kwargs, T, **kw):
    """Anchors x_{t,0} for t = 0..T and the mean directions, by running prefixes."""
    xs = [np.full(N, f32(cfg_kwargs.get("x_init", 0.0)))]
    us = [np.zeros(N)]
    last = None
    for t in range(1, T + 1):
        c = oracle.make_config(T=t, **cfg_kwargs)
        g = kw.get("gamma_t")
        last = run64(c, want_dbar=True, gamma_t=None if g is None else g[:t])
        xs.append(last["anchor"])
        us.append(last["u"])
    return xs, us, last["dbar"]


@pytest.mark.parametrize("base", ["nesterov", "adam"])
def test_equivalent_update_identities(base):
    kw = dict(m=4, tau=5, alpha=0.8, beta=0.6, gamma=0.03, base=base, mu=0.9, sigma=0.2, seed=8,
              adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, buffer_policy="maintain", x_init=0.3)
    T = 6
    xs, us, dbar = _anchors(kw, T)
    alpha, beta, gam = f32(0.8), f32(0.6), f32(0.03)
    D = dbar.sum(axis=1)  # sum_k dbar_{t,k}
    for t in range(T):
        # x_{t+1,0} = x_{t,0} - alpha gamma sum_k dbar + beta (x_{t,0} - x_{t-1,0})
        prev = xs[t] - xs[t - 1] if t > 0 else 0.0
        close(xs[t + 1], xs[t] - alpha * gam * D[t] + beta * prev, 1e-11)
        # u_{t+1} = beta u_t + sum_k dbar  (the average is x_{t,0} - gamma sum_k dbar)
        close(us[t + 1], beta * us[t] + D[t], 1e-10)
    # auxiliary sequence y_t = x_t + beta/(1-beta) (x_t - x_{t-1}) moves by -alpha gamma/(1-beta) sum_k dbar
    y = [xs[0]] + [xs[t] + beta / (1 - beta) * (xs[t] - xs[t - 1]) for t in range(1, T + 1)]
    for t in range(T):
        close(y[t + 1], y[t] - alpha * gam / (1 - beta) * D[t], 1e-10)
    # x_t - x_{t-1} = -alpha gamma sum_{s<t} beta^{t-1-s} sum_k dbar_{s,k}
    for t in range(1, T + 1):
        acc = sum(beta ** (t - 1 - s) * D[s] for s in range(t))
        close(xs[t] - xs[t - 1], -alpha * gam * acc, 1e-11)


def test_slow_momentum_is_invariant_to_the_base_learning_rate_schedule():
    # with gamma_t changing between outer iterations u still obeys u_{t+1} = beta u_t + sum_k dbar_{t,k}
    kw = dict(m=3, tau=4, alpha=1.0, beta=0.7, gamma=0.05, mu=0.9, sigma=0.1, seed=9)
    T = 5
    gammas = np.array([0.01, 0.05, 0.1, 0.02, 0.004], np.float32)
    xs, us, dbar = _anchors(kw, T, gamma_t=gammas)
    beta = f32(0.7)
    D = dbar.sum(axis=1)
    for t in range(T):
        close(us[t + 1], beta * us[t] + D[t], 1e-9)
        close(xs[t + 1], xs[t] - 1.0 * float(gammas[t]) * us[t + 1], 1e-11)


def test_all_workers_hold_the_anchor_after_an_outer_step():
    for prec in ("f32", "f64"):
        for base, policy in itertools.product(("nesterov", "adam"), ("reset", "maintain", "average")):
            cfg = oracle.make_config(m=5, tau=3, T=4, alpha=0.9, beta=0.5, gamma=0.02, base=base, mu=0.9,
                                     sigma=0.1, buffer_policy=policy, seed=10)
            out = oracle.run(cfg, j0=0, n=N, precision=prec)
            for i in range(5):
                assert np.array_equal(out["x"][i], out["anchor"])
            if policy == "reset":
                assert not out["h"].any() and not out["v"].any()
            if policy == "average":
                assert all(np.array_equal(out["h"][i], out["h"][0]) for i in range(5))


# -------------------------------------------------------------------------- closed forms

@pytest.mark.parametrize("mu,wd", [(0.9, 0.0), (0.9, 1e-2), (0.0, 0.0)])
def test_noise_free_quadratic_closed_form(mu, wd):
    # sigma = 0, buffers reset. Per worker, with a' = a + wd and c' = a c / a', the pair
    # (e, h) = (x - c', h) obeys a 2x2 linear map M per step; from e_0 = E, h_0 = 0 the
    # first component after tau steps is rho E (rho = (M^tau)_00, the same for all workers),
    # so the average error contracts by rho and (E_t, gamma u_t) follow a second 2x2 map.
    tau, T, m = 7, 6, 4
    cfg = oracle.make_config(m=m, tau=tau, T=T, alpha=0.9, beta=0.6, gamma=0.05, mu=mu, sigma=0.0,
                             weight_decay=wd, buffer_policy="reset", seed=11, x_init=0.25)
    p = Problem(cfg)
    gam, mu_, wd_, alpha, beta = f32(0.05), f32(mu), f32(wd), f32(0.9), f32(0.6)
    out = run64(cfg)
    for q in range(N):
        a1 = p.a[q] + wd_
        cbar = np.mean(p.a[q] * p.c[:, q] / a1)
        M = np.array([[1 - gam * a1 * (1 + mu_), -gam * mu_ * mu_], [a1, mu_]])
        rho = np.linalg.matrix_power(M, tau)[0, 0]
        Nmat = np.array([[1 - alpha * (1 - rho), -alpha * beta], [1 - rho, beta]])
        E, w = np.linalg.matrix_power(Nmat, T) @ np.array([f32(0.25) - cbar, 0.0])
        assert abs(out["anchor"][q] - (E + cbar)) < 1e-12
        assert abs(out["u"][q] * gam - w) < 1e-12


def test_adam_first_step_is_sign_like():
    # with zero buffers the first Adam direction is g / (|g| + eps): every bias correction cancels
    cfg = oracle.make_config(m=2, tau=1, T=1, alpha=1.0, beta=0.0, gamma=0.01, base="adam", sigma=0.5,
                             adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, buffer_policy="maintain", seed=12)
    p = Problem(cfg)
    out = run64(cfg, want_dbar=True)
    g = np.stack([p.grad(0, 0, i, np.zeros(N)) for i in range(2)])
    d = g / (np.abs(g) + f32(1e-8))
    close(out["dbar"][0, 0], d.mean(axis=0), 1e-6)  # bias-correction constants are rounded to binary64 once
    close(out["anchor"], -f32(0.01) * d.mean(axis=0), 1e-6)


# ---------------------------------------------------------------------- library optimizers

def _torch_trajectory(opt_factory, p, steps_t, tau):
    x = torch.zeros(N, dtype=torch.float64, requires_grad=True)
    opt = opt_factory([x])
    for t in range(steps_t):
        for k in range(tau):
            opt.zero_grad()
            # gradient without weight decay: the optimizer adds its own L2 term
            g = p.a * (x.detach().numpy() - p.c[0]) + p.sigma * p.z(t, k, 0)
            x.grad = torch.from_numpy(g.copy())
            opt.step()
    return x.detach().numpy()


def test_single_replica_nesterov_matches_torch_sgd():
    # m = 1, alpha = 1, beta = 0, buffers maintained: the outer step is the identity and the
    # run is plain Nesterov SGD with L2 weight decay
    wd = 1e-3
    cfg = oracle.make_config(m=1, tau=5, T=8, alpha=1.0, beta=0.0, gamma=0.05, mu=0.9, sigma=0.2,
                             weight_decay=wd, buffer_policy="maintain", seed=13)
    p = Problem(cfg)
    ref = _torch_trajectory(lambda ps: torch.optim.SGD(ps, lr=f32(0.05), momentum=f32(0.9), nesterov=True,
                                                      weight_decay=f32(wd)), p, 8, 5)
    close(run64(cfg)["anchor"], ref, 1e-12)


def test_single_replica_adam_matches_torch_adam():
    cfg = oracle.make_config(m=1, tau=6, T=7, alpha=1.0, beta=0.0, gamma=5e-3, base="adam", sigma=0.2,
                             adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, buffer_policy="maintain", seed=14)
    p = Problem(cfg)
    ref = _torch_trajectory(lambda ps: torch.optim.Adam(ps, lr=f32(5e-3), betas=(f32(0.9), f32(0.98)),
                                                       eps=f32(1e-8)), p, 7, 6)
    # torch divides sqrt(v) by sqrt(1-b2^l) and h by (1-b1^l); same value, other rounding order
    close(run64(cfg)["anchor"], ref, 1e-9)


# ------------------------------------------------------------------------------ brute force

class _Worker:
    """One worker of Algorithm 1 with its own parameter, buffers and step counter."""

    def __init__(self, x0, hp):
        self.x, self.h, self.v, self.l, self.hp = x0, 0.0, 0.0, 0, hp

    def step(self, g, gam):
        hp = self.hp
        if hp["base"] == "nesterov":
            self.h = hp["mu"] * self.h + g
            d = hp["mu"] * self.h + g
        else:
            self.l += 1
            self.h = hp["b1"] * self.h + (1 - hp["b1"]) * g
            self.v = hp["b2"] * self.v + (1 - hp["b2"]) * g * g
            hh = self.h / (1 - hp["b1"] ** self.l)
            vh = self.v / (1 - hp["b2"] ** self.l)
            d = hh / (np.sqrt(vh) + hp["eps"])
        self.x = self.x - gam * d


@pytest.mark.parametrize("base,policy", list(itertools.product(("nesterov", "adam"),
                                                               ("reset", "maintain", "average"))))
@pytest.mark.parametrize("m", [1, 3, 5])
def test_brute_force_with_worker_objects_and_averaging_matrix(base, policy, m):
    tau, T, n = 3, 4, 6
    kw = dict(m=m, tau=tau, T=T, alpha=0.75, beta=0.4, gamma=0.02 if base == "adam" else 0.08, base=base,
              mu=0.8, sigma=0.3, weight_decay=2e-3, adam_b1=0.9, adam_b2=0.95, adam_eps=1e-6,
              buffer_policy=policy, seed=20 + m, x_init=-0.2)
    cfg = oracle.make_config(**kw)
    p = Problem(cfg, n)
    hp = dict(base=base, mu=f32(0.8), b1=f32(0.9), b2=f32(0.95), eps=f32(1e-6))
    gam, alpha, beta = f32(kw["gamma"]), f32(0.75), f32(0.4)
    W = np.full((m, m), 1.0 / m)  # exact-averaging matrix (1/m) 1 1^T
    out = oracle.run(cfg, j0=0, n=n, precision="f64")
    for q in range(n):
        workers = [_Worker(f32(-0.2), hp) for _ in range(m)]
        anchor, u = f32(-0.2), 0.0
        for t in range(T):
            for k in range(tau):
                for i, wk in enumerate(workers):
                    z = float(p.z(t, k, i)[q])
                    g = p.a[q] * (wk.x - p.c[i, q]) + p.sigma * z + p.wd * wk.x
                    wk.step(g, gam)
            xbar = (W @ np.array([wk.x for wk in workers]))[0]
            u = beta * u + (anchor - xbar) / gam
            anchor = anchor - alpha * gam * u
            for wk in workers:
                wk.x = anchor
            if policy == "reset":
                for wk in workers:
                    wk.h, wk.v, wk.l = 0.0, 0.0, 0
            elif policy == "average":
                hb = (W @ np.array([wk.h for wk in workers]))[0]
                vb = (W @ np.array([wk.v for wk in workers]))[0]
                for wk in workers:
                    wk.h, wk.v = hb, vb
        assert abs(out["anchor"][q] - anchor) < 1e-11 * (1 + abs(anchor))
        assert abs(out["u"][q] - u) < 1e-10 * (1 + abs(u))
        for i, wk in enumerate(workers):
            assert abs(out["h"][i, q] - wk.h) < 1e-11 * (1 + abs(wk.h))
            assert abs(out["v"][i, q] - wk.v) < 1e-11 * (1 + abs(wk.v))


def test_supplied_gradient_modes():
    # supplied array: direction does not depend on x; with plain SGD the run telescopes
    m, tau, T, n = 3, 4, 3, 10
    from paper_1910_00643_b200.workloads import dense_gradients
    G = dense_gradients(T * tau, m, n, seed=3)
    cfg = oracle.make_config(m=m, tau=tau, T=T, alpha=1.0, beta=0.0, gamma=0.1, mu=0.0,
                             grad_mode="supplied_array", buffer_policy="reset")
    out = oracle.run(cfg, j0=0, n=n, precision="f64", G=G)
    close(out["anchor"], -f32(0.1) * G.astype(np.float64).mean(axis=1).sum(axis=0), 1e-12)
    # supplied hash: the same gradient sigma z(tag 5) at every step
    cfg = oracle.make_config(m=m, tau=tau, T=1, alpha=1.0, beta=0.0, gamma=0.1, mu=0.0, sigma=0.1,
                             grad_mode="supplied", seed=4)
    out = oracle.run(cfg, j0=5, n=n, precision="f64")
    g = np.stack([oracle.supplied_gradient(cfg, i, np.arange(5, 5 + n)) for i in range(m)]).astype(np.float64)
    close(out["anchor"], -f32(0.1) * tau * g.mean(axis=0), 1e-12)


# ------------------------------------------------------------------ binary32 mode vs binary64

def test_binary32_mode_tracks_binary64_mode():
    for kw in (dict(m=4, tau=4, T=3, alpha=1.0, beta=0.6, gamma=0.05, mu=0.9, sigma=0.1),
               dict(m=8, tau=12, T=4, alpha=1.0, beta=0.7, gamma=0.1, mu=0.9, weight_decay=1e-4,
                    a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.01, buffer_policy="average")):
        cfg = oracle.make_config(**kw)
        a = oracle.run(cfg, j0=0, n=4096, precision="f32")
        b = oracle.run(cfg, j0=0, n=4096, precision="f64")
        for key in ("x", "anchor", "u", "h"):
            err = np.abs(a[key].astype(np.float64) - b[key])
            assert (err <= 1e-5 * (1 + np.abs(b[key]))).all(), (key, err.max())


def test_coordinate_lists_and_ranges_agree():
    cfg = oracle.make_config(m=3, tau=2, T=2, beta=0.5, gamma=0.05, mu=0.9, sigma=0.1)
    full = oracle.run(cfg, j0=0, n=100)
    pick = np.array([99, 0, 17, 17, 42], np.uint64)
    some = oracle.run(cfg, j=pick)
    assert np.array_equal(some["x"], full["x"][:, pick.astype(int)])
    assert np.array_equal(some["u"], full["u"][pick.astype(int)])


def test_binary32_oracle_matches_its_frozen_outputs():
    # regression net: the stored bit patterns were written by tests/golden/make_oracle_golden.py from
    # the oracle itself; a mismatch means the oracle's arithmetic changed
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(__file__), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(here, "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = [l.strip() for l in open(os.path.join(here, "oracle_f32_cases.txt")) if not l.startswith("#")]
    assert stored == list(mod.lines())
