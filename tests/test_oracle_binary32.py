"""Pins for the binary32 instantiation of the oracle (the parity gate) beyond the Nesterov cases:
Adam (Table C.1, Adam row), the SGP bases (Algorithm 2; Table C.1, SGP rows) and the variant
without the exact average (Section 6 of the paper).

Two things are checked for each case, on tens of thousands of coordinates:

  1. the binary64 mode agrees (1e-11) with a float64 restatement written here with whole-array
     numpy operations (one array per worker, explicit row rotation for the push-sum mixing, numpy
     means for the averages) -- a second, differently structured implementation on the generated
     gradient, which the single-replica torch.optim pins do not cover;
  2. the binary32 mode stays within the parity tolerance 1e-5 (1 + |s|) of the binary64 mode, except
     where Adam's direction is ill-conditioned: d = h_hat / (sqrt(v_hat) + eps) with eps = 1e-8 is
     close to sign(g) while v_hat is still made of one or two gradients, so an element whose gradient
     is tiny (|g| < 1e-6) while sqrt(v_hat) is tiny (< 1e-5) at some step turns rounding error into
     an O(gamma) change of x. Such elements are counted and must be the ONLY ones outside the
     tolerance; they are never silently dropped.

A slip that exists only in the binary32 build (a float-only constant, sqrt in place of sqrtf's
rounding, a missing cast) shows up in 2 on well-conditioned elements.
"""
import numpy as np
import pytest

import oracle

RTOL = 1e-5


def f32(v):
    return float(np.float32(v))


def restatement(kw, n):
    """Algorithm 1 in float64 with one numpy array per quantity and worker axis first. Returns the
    final state and, per coordinate, whether any worker met the ill-conditioning criterion."""
    cfg = oracle.make_config(**kw)
    m, tau, T = kw["m"], kw["tau"], kw["T"]
    j = np.arange(n)
    a = oracle.curvature(cfg, j).astype(np.float64)
    c = np.stack([oracle.centre(cfg, i, j) for i in range(m)]).astype(np.float64)
    sig, wd = f32(kw.get("sigma", 0.0)), f32(kw.get("weight_decay", 0.0))
    gam, alpha, beta = f32(kw["gamma"]), f32(kw.get("alpha", 1.0)), f32(kw.get("beta", 0.0))
    b1, b2, eps = f32(kw.get("adam_b1", 0.9)), f32(kw.get("adam_b2", 0.999)), f32(kw.get("adam_eps", 1e-8))
    mu = f32(kw.get("mu", 0.0))
    base = kw.get("base", "nesterov")
    adam, sgp, noavg = "adam" in base, base.startswith("sgp"), kw.get("no_average", False)
    policy = kw.get("buffer_policy", "reset")
    x = np.full((m, n), f32(kw.get("x_init", 0.0)))
    h, v = np.zeros((m, n)), np.zeros((m, n))
    anchor = x.copy() if noavg else x[0].copy()
    u = np.zeros_like(anchor)
    steps_since_zero = 0
    ill = np.zeros(n, bool)
    for t in range(T):
        for k in range(tau):
            steps_since_zero += 1
            z = np.stack([oracle.stream(oracle.TAG_GRADNOISE, cfg.seed, t, k, i, 0, n, words=False)[1]
                          for i in range(m)]).astype(np.float64)
            g = a * (x - c) + sig * z + wd * x
            if adam:
                h = b1 * h + (1 - b1) * g
                v = b2 * v + (1 - b2) * g * g
                root = np.sqrt(v / (1 - b2 ** steps_since_zero))
                d = (h / (1 - b1 ** steps_since_zero)) / (root + eps)
                ill |= ((np.abs(g) < 1e-6) & (root < 1e-5)).any(axis=0)
            else:
                h = mu * h + g
                d = mu * h + g
            x = x - gam * d
            if sgp and m > 1:
                # keep half, receive half from the worker `hops` places back
                x = 0.5 * x + 0.5 * np.roll(x, oracle.sgp_hops(m, t * tau + k), axis=0)
        if noavg:
            u = beta * u + (anchor - x) / gam
            anchor = anchor - alpha * gam * u
            x = anchor.copy()
        else:
            u = beta * u + (anchor - x.mean(axis=0)) / gam
            anchor = anchor - alpha * gam * u
            x = np.tile(anchor, (m, 1))
        if policy == "reset":
            h[:], v[:], steps_since_zero = 0.0, 0.0, 0
        elif policy == "average":
            h[:], v[:] = h.mean(axis=0), v.mean(axis=0)
    return {"x": x, "h": h, "v": v, "anchor": anchor, "u": u}, ill


ADAM = dict(adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8)
CASES = {
    # the transformer-shaped workload's hyperparameters (Local Adam, buffers kept)
    "adam-maintain": dict(m=8, tau=12, T=5, alpha=1.0, beta=0.5, gamma=5e-4, base="adam", a_lo=0.1, a_hi=1.0,
                          c_std=0.02, sigma=0.01, buffer_policy="maintain", **ADAM),
    "adam-reset-wd": dict(m=4, tau=3, T=4, alpha=0.9, beta=0.6, gamma=0.01, base="adam", sigma=0.1,
                          buffer_policy="reset", weight_decay=1e-3, **ADAM),
    "adam-average": dict(m=4, tau=3, T=4, alpha=0.9, beta=0.6, gamma=0.01, base="adam", sigma=0.05,
                         buffer_policy="average", x_init=-0.5, **ADAM),
    "sgp-adam-maintain": dict(m=5, tau=4, T=3, alpha=0.9, beta=0.6, gamma=0.01, base="sgp_adam", sigma=0.1,
                              buffer_policy="maintain", **ADAM),
    "sgp-adam-reset": dict(m=8, tau=5, T=3, alpha=1.0, beta=0.5, gamma=5e-4, base="sgp_adam", a_lo=0.1, a_hi=1.0,
                           c_std=0.02, sigma=0.01, buffer_policy="reset", **ADAM),
    "sgp-nesterov-reset": dict(m=6, tau=5, T=3, alpha=1.0, beta=0.6, gamma=0.05, mu=0.9, base="sgp_nesterov",
                               sigma=0.1, buffer_policy="reset", weight_decay=1e-4),
    "sgp-nesterov-average": dict(m=7, tau=6, T=2, alpha=1.0, beta=0.6, gamma=0.1, mu=0.9, base="sgp_nesterov",
                                 a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.01, buffer_policy="average",
                                 weight_decay=1e-4),
    "noaverage-adam": dict(m=3, tau=4, T=3, alpha=0.9, beta=0.6, gamma=0.01, base="adam", sigma=0.1,
                           buffer_policy="maintain", no_average=True, **ADAM),
    "noaverage-nesterov": dict(m=4, tau=4, T=3, alpha=0.9, beta=0.6, gamma=0.05, mu=0.9, base="nesterov",
                               sigma=0.1, buffer_policy="reset", no_average=True),
    "noaverage-sgp-nesterov": dict(m=4, tau=4, T=3, alpha=0.9, beta=0.6, gamma=0.05, mu=0.9, base="sgp_nesterov",
                                   sigma=0.1, buffer_policy="maintain", no_average=True),
}


def _compare(kw, n):
    cfg = oracle.make_config(**kw)
    lo = oracle.run(cfg, j0=0, n=n, precision="f32")
    hi = oracle.run(cfg, j0=0, n=n, precision="f64")
    ref, ill = restatement(kw, n)
    keys = ["x", "anchor", "u", "h"] + (["v"] if "adam" in kw["base"] else [])
    outside = np.zeros(n, bool)
    for key in keys:
        # 1: the binary64 mode against the restatement
        gap = np.abs(hi[key] - ref[key]) / (1.0 + np.abs(ref[key]))
        assert gap.max() < 1e-11 or ill.any(), (key, gap.max())
        assert gap.reshape(-1, n)[:, ~ill].max() < 1e-11, (key, gap.max())
        # 2: the binary32 mode against the binary64 mode
        err = np.abs(lo[key].astype(np.float64) - hi[key])
        outside |= (err > RTOL * (1.0 + np.abs(hi[key]))).reshape(-1, n).any(axis=0)
    return outside, ill


@pytest.mark.parametrize("name", sorted(CASES))
def test_binary32_mode_is_within_tolerance_of_binary64_mode_except_where_adam_is_ill_conditioned(name):
    n = 20_000
    outside, ill = _compare(CASES[name], n)
    # every element outside the tolerance is an ill-conditioned one; those are few
    assert not (outside & ~ill).any(), f"{int((outside & ~ill).sum())} well-conditioned coordinates outside tolerance"
    assert ill.sum() <= n // 100, int(ill.sum())
    if "adam" not in CASES[name]["base"]:
        assert not ill.any() and not outside.any()


@pytest.mark.parametrize("extra", [dict(base="adam", buffer_policy="reset"),
                                   dict(base="adam", buffer_policy="maintain", no_average=True)])
def test_the_ill_conditioning_criterion_explains_every_element_outside_the_tolerance(extra):
    # a regime made to hit the criterion often: gradients of order 1e-4, so |g| < 1e-6 while v_hat
    # is still one or two tiny gradients happens for a few per cent of the coordinates
    kw = dict(m=4, tau=3, T=4, alpha=0.9, beta=0.6, gamma=0.01, sigma=1e-4, c_std=1e-4, a_lo=0.1, a_hi=1.0,
              **ADAM, **extra)
    n = 100_000
    outside, ill = _compare(kw, n)
    assert outside.sum() > 20, "the regime no longer produces ill-conditioned elements: the test is vacuous"
    assert not (outside & ~ill).any(), int((outside & ~ill).sum())
    assert ill.sum() < n // 10
