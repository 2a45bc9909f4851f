"""Seeded synthetic workloads: problem sizes, hyperparameters and input tensors.

This module only describes inputs. It holds none of the method's arithmetic and imports
neither the CUDA binding nor the CPU oracle, so the same description can be handed to both.

The workloads stand in for the paper's training jobs, whose datasets and models are not
available: only shapes and hyperparameters are taken from the paper (Section 4 and
Appendix A: ResNet-50 on ImageNet with m = 32 nodes, tau = 12, beta = 0.7, Nesterov
momentum 0.9, weight decay 1e-4; transformer-big on WMT'16 with m = 8 nodes, Adam
(0.9, 0.98, 1e-8), buffers maintained). The per-worker objective is the separable quadratic
F_i(x) = 1/2 sum_j a_j (x_j - c_{i,j})^2 with hash-generated gradient noise.

Keys of a workload dict (paper notation): P parameters, m workers, tau inner steps, T outer
iterations, alpha / beta slow learning rate and momentum, gamma base learning rate, base
optimizer and its constants, buffer_policy (first statement of Algorithm 1's outer loop),
grad_mode, and the generator constants seed, a_lo, a_hi, c_std, sigma, x_init.
"""
import numpy as np

_QUADRATIC_SMALL = dict(a_lo=0.5, a_hi=2.0, c_std=1.0, sigma=0.1, seed=0, x_init=0.0)
_NESTEROV_SMALL = dict(base="nesterov", gamma=0.05, mu=0.9, weight_decay=0.0)

WORKLOADS = {
    # tiny SlowMo on a noisy separable quadratic
    "tiny": dict(P=4096, m=4, tau=4, T=3, alpha=1.0, beta=0.6, buffer_policy="reset",
                 grad_mode="generated", **_NESTEROV_SMALL, **_QUADRATIC_SMALL),
    # ResNet-50-shaped replica set (Local SGD + SlowMo on ImageNet in the paper)
    "resnet50": dict(P=25_557_032, m=32, tau=12, T=10, alpha=1.0, beta=0.7,
                     buffer_policy="average", grad_mode="generated", base="nesterov", gamma=0.1,
                     mu=0.9, weight_decay=1e-4, a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.01,
                     seed=0, x_init=0.0, n_tensors=161),
    # BMUF-style run and the two degenerate cases of Section 2
    "bmuf": dict(P=25_557_032, m=16, tau=48, T=5, alpha=1.0, beta=0.5, buffer_policy="reset",
                 grad_mode="generated", **_NESTEROV_SMALL, **_QUADRATIC_SMALL),
    "local_sgd": dict(P=25_557_032, m=16, tau=48, T=5, alpha=1.0, beta=0.0,
                      buffer_policy="reset", grad_mode="generated", **_NESTEROV_SMALL,
                      **_QUADRATIC_SMALL),
    "sync_sgd": dict(P=25_557_032, m=16, tau=1, T=5, alpha=1.0, beta=0.0,
                     buffer_policy="average", grad_mode="generated", **_NESTEROV_SMALL,
                     **_QUADRATIC_SMALL),
    # transformer-big-shaped replica set with Adam (Local Adam + SlowMo on WMT'16)
    "transformer_adam": dict(P=210_000_000, m=8, tau=12, T=5, alpha=1.0, beta=0.5,
                             buffer_policy="maintain", grad_mode="generated", base="adam",
                             gamma=5e-4, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8,
                             weight_decay=0.0, a_lo=0.1, a_hi=1.0, c_std=0.02, sigma=0.01,
                             seed=0, x_init=0.0),
    # stochastic gradient push as the base optimizer (the paper's SGP + SlowMo on ImageNet: tau = 48,
    # Nesterov buffers zeroed at each outer step) and its Adam form (WMT'16)
    "sgp_resnet50": dict(P=25_557_032, m=32, tau=48, T=3, alpha=1.0, beta=0.6, buffer_policy="reset",
                         grad_mode="generated", base="sgp_nesterov", gamma=0.1, mu=0.9, weight_decay=1e-4,
                         a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.01, seed=0, x_init=0.0),
    "sgp_transformer_adam": dict(P=210_000_000, m=8, tau=48, T=2, alpha=1.0, beta=0.5,
                                 buffer_policy="maintain", grad_mode="generated", base="sgp_adam",
                                 gamma=5e-4, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, weight_decay=0.0,
                                 a_lo=0.1, a_hi=1.0, c_std=0.02, sigma=0.01, seed=0, x_init=0.0),
    # bandwidth stress: supplied gradient tensor, tau swept over {1, 12, 48}
    "stress_tau1": dict(P=1_000_000_000, m=4, tau=1, T=3, alpha=1.0, beta=0.6,
                        buffer_policy="reset", grad_mode="supplied", sigma=0.1, seed=0,
                        x_init=0.0, **_NESTEROV_SMALL),
    "stress_tau12": dict(P=1_000_000_000, m=4, tau=12, T=3, alpha=1.0, beta=0.6,
                         buffer_policy="reset", grad_mode="supplied", sigma=0.1, seed=0,
                         x_init=0.0, **_NESTEROV_SMALL),
    "stress_tau48": dict(P=1_000_000_000, m=4, tau=48, T=3, alpha=1.0, beta=0.6,
                         buffer_policy="reset", grad_mode="supplied", sigma=0.1, seed=0,
                         x_init=0.0, **_NESTEROV_SMALL),
}


def workload(name, **overrides):
    """A copy of a named workload with optional overrides (e.g. a smaller P for a test)."""
    w = dict(WORKLOADS[name])
    w.update(overrides)
    w["name"] = name
    return w


def tensor_sizes(P, n_tensors, seed=0, span_log2=15):
    """Split P into n_tensors segment sizes drawn log-uniformly over a 2^span_log2 range.

    A log-uniform size has density proportional to 1/s, i.e. a power law: a few large
    tensors hold most parameters and many small ones (biases, norms) hold few, as in a
    convolutional network. Sizes are positive and sum to P exactly; the remainder of the
    rounding goes to the largest segment. This is metadata only: kernels see one flat vector.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    w = np.exp(rng.random(n_tensors) * np.log(2.0 ** span_log2))
    sizes = np.maximum(1, np.floor(P * w / w.sum())).astype(np.uint64)
    big = int(np.argmax(sizes))
    rest = int(P) - int(sizes.sum())
    assert int(sizes[big]) + rest >= 1
    sizes[big] = np.uint64(int(sizes[big]) + rest)
    return sizes


def dense_gradients(steps, m, n, seed=0, scale=1.0):
    """A seeded [steps, m, n] float32 tensor of arbitrary gradients for supplied-gradient tests."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return (scale * rng.standard_normal((steps, m, n))).astype(np.float32)


def sample_coordinates(P, count, seed=0, tile=4096):
    """Coordinates at which a full-size run is compared with the oracle.

    Both ends of the vector, both sides of tile boundaries near the start, the middle and
    the end, and uniformly drawn coordinates; sorted and unique.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    edges = [np.arange(0, min(P, 64)), np.arange(max(0, P - 64), P)]
    for b in (tile, (P // 2 // tile) * tile, (P // tile) * tile):
        lo, hi = max(0, b - 16), min(P, b + 16)
        if lo < hi:
            edges.append(np.arange(lo, hi))
    rand = rng.integers(0, P, size=max(0, count), dtype=np.int64)
    j = np.unique(np.concatenate(edges + [rand]).astype(np.uint64))
    return j
