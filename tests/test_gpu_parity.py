"""GPU parity: the CUDA library (through its C ABI) against the binary32 oracle, element by
element on small cases and on sampled coordinates at the full benchmark sizes.

Gate (all state tensors x, anchor, u, h, v after the full run):
    max |gpu - oracle| <= 1e-5 * (1 + |oracle|)
The integer noise stream must match bit for bit.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_1910_00643_b200 import workloads

pytestmark = pytest.mark.gpu

RTOL = 1e-5


def _slowmo(w, **kw):
    from paper_1910_00643_b200 import SlowMo
    return SlowMo(w, **kw)


def _state_keys(w):
    return ("x", "anchor", "u", "h") + (("v",) if "adam" in w.get("base", "") else ())


def _gather(s, key, j):
    """Columns j of a state tensor, straight from device memory."""
    import torch
    idx = torch.as_tensor(np.asarray(j, dtype=np.int64), device="cuda")
    t = s.t[key]
    two_d = key in ("x", "h", "v", "c") or (key in ("anchor", "u") and s.cfg.no_average)
    out = t.view(s.m if two_d else 1, s.pitch).index_select(1, idx).cpu().numpy()
    return out if two_d else out[0]


def _assert_close(got, ref, what):
    got64, ref64 = got.astype(np.float64), ref.astype(np.float64)
    err = np.abs(got64 - ref64)
    bad = err > RTOL * (1.0 + np.abs(ref64))
    assert not bad.any(), f"{what}: {int(bad.sum())} elements off, max |d| = {err.max():.3e}"
    assert np.isfinite(got64).all(), what


def _check_against_oracle(s, w, j, T=None, gamma_t=None, G=None, exact=False):
    s.sync_status()
    cfg = oracle.make_config(**dict(w, T=w["T"] if T is None else T))
    ref = oracle.run(cfg, j=np.asarray(j, np.uint64), precision="f32", gamma_t=gamma_t, G=G)
    for key in _state_keys(w):
        got = _gather(s, key, j)
        _assert_close(got, ref[key], f"{w.get('name')}:{key}")
        if exact:
            assert np.array_equal(got.view(np.uint32), ref[key].view(np.uint32)), f"{key} not bit-equal"
    return ref


# ------------------------------------------------------------------------------- noise stream

def test_noise_words_and_normals_are_bit_exact():
    s = _slowmo(workloads.workload("tiny", seed=77))
    cases = [(3, 0, 0, 0, 0), (3, 2, 3, 1, 12345), (1, 0, 0, 0, 0), (2, 0, 0, 3, 999), (5, 0, 0, 2, 7),
             (3, 2**40 + 5, 47, 31, 2**32 - 100), (3, 9, 1, 0, 2**33 + 1)]
    for tag, t, k, wk, j0 in cases:
        n = 5000
        gw, gz = s.debug_noise(tag, t, k, wk, j0, n)
        ow, oz = oracle.stream(tag, 77, t, k, wk, j0, n)
        assert np.array_equal(gw, ow), (tag, t, k, wk, j0)
        assert np.array_equal(gz.view(np.uint32), oz.view(np.uint32)), (tag, t, k, wk, j0)
    s.close()


def test_normals_bit_exact_on_a_large_sample():
    s = _slowmo(workloads.workload("tiny"))
    n = 1 << 22
    gw, gz = s.debug_noise(3, 1, 2, 3, 0, n)
    ow, oz = oracle.stream(3, 0, 1, 2, 3, 0, n)
    assert np.array_equal(gw, ow)
    assert np.array_equal(gz.view(np.uint32), oz.view(np.uint32))
    s.close()


def test_normal_map_is_bit_exact_for_every_radius_field_and_every_angle_field():
    # z = radius(k1) * trig(k2) with an IEEE multiply, so agreement for all 2^24 values of each field
    # (with the other field fixed) gives agreement for every word
    s = _slowmo(workloads.workload("tiny"))
    all24 = np.arange(1 << 24, dtype=np.uint64)
    for words in (all24 << np.uint64(40),                                   # every k1, angle 0: zc = radius
                  (all24 << np.uint64(40)) | np.uint64(0x1234560000),       # every k1, a generic angle
                  all24 << np.uint64(16),                                   # every k2, largest radius
                  (np.uint64(0x5A5A5A) << np.uint64(40)) | (all24 << np.uint64(16)) | np.uint64(0xBEEF)):
        got = s.debug_words_to_normals(words)
        ref = oracle.words_to_normals(words)
        assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    s.close()


def test_problem_data_fill_matches_oracle():
    w = workloads.workload("tiny", P=5003, m=3, a_lo=0.1, a_hi=1.0, c_std=0.05, seed=5)
    s = _slowmo(w, guard=64)
    cfg = oracle.make_config(**w)
    j = np.arange(w["P"])
    a = s.get_params("a")[0]
    assert np.array_equal(a.view(np.uint32), oracle.curvature(cfg, j).view(np.uint32))
    c = s.get_params("c")
    for i in range(3):
        assert np.array_equal(c[i].view(np.uint32), oracle.centre(cfg, i, j).view(np.uint32))
    x = s.get_params("x")
    assert (x == np.float32(w["x_init"])).all() and not s.get_params("u").any() and not s.get_params("h").any()
    assert s.guards_intact()
    s.close()


def test_supplied_gradient_fill_matches_oracle():
    w = workloads.workload("stress_tau1", P=4099, m=2, sigma=0.3, seed=11)
    s = _slowmo(w, guard=64)
    g = s.alloc_gradient()
    s.fill_gradient()
    s.synchronize()
    cfg = oracle.make_config(**w)
    got = g.view(2, s.pitch)[:, :w["P"]].cpu().numpy()
    for i in range(2):
        ref = oracle.supplied_gradient(cfg, i, np.arange(w["P"]))
        assert np.array_equal(got[i].view(np.uint32), ref.view(np.uint32))
    assert s.guards_intact()
    s.close()


# ------------------------------------------------------------- small cases, element by element

SMALL_P = 3 * 1024 + 37  # several 512- and 1024-column tiles and a ragged tail (not a multiple of 4)


@pytest.mark.parametrize("variant", ["direct", "staged", "fused", "lazy"])
@pytest.mark.parametrize("base,policy", list(itertools.product(("nesterov", "adam"), ("reset", "maintain", "average"))))
@pytest.mark.parametrize("m", [1, 3, 4, 9])
def test_small_runs_match_oracle(base, policy, m, variant):
    w = workloads.workload("tiny", P=SMALL_P, m=m, tau=3, T=3, base=base, buffer_policy=policy, alpha=0.9,
                           beta=0.6, gamma=0.01 if base == "adam" else 0.05, weight_decay=1e-3,
                           adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, seed=3)
    s = _slowmo(w, guard=64)
    s.set_variant("outer", variant)
    s.run(w["T"])
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    assert s.counters()[0] == 3 and s.counters()[1] == 0
    s.close()


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 511, 512, 513, 1023, 1024, 1025, 2048 + 4])
def test_ragged_sizes(P):
    w = workloads.workload("tiny", P=P, m=5, tau=2, T=2, buffer_policy="average")
    for variant in ("direct", "staged", "fused", "lazy"):
        s = _slowmo(w, guard=64)
        s.set_variant("outer", variant)
        s.run(2)
        _check_against_oracle(s, w, np.arange(P), exact=True)
        assert s.guards_intact()
        s.close()


def test_tiny_workload_full_run():
    w = workloads.workload("tiny")
    s = _slowmo(w)
    s.run(w["T"])
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    s.close()


def test_many_workers():
    w = workloads.workload("tiny", P=2051, m=32, tau=2, T=2, buffer_policy="average")
    for variant in ("direct", "staged", "fused", "lazy"):
        s = _slowmo(w)
        s.set_variant("outer", variant)
        s.run(2)
        _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
        s.close()


@pytest.mark.parametrize("layout", ["default", "row_tiles", "column_owner"])
@pytest.mark.parametrize("variant", ["direct", "staged", "fused", "lazy"])
def test_more_workers_than_inline_noise_keys(variant, layout):
    # beyond 64 workers the noise keys no longer travel in the kernel arguments: the kernels derive
    # them (one lane per warp in the row-tile layout, 32 rows per warp pass in the column-owner ones)
    w = workloads.workload("tiny", P=1030, m=70, tau=3, T=2, buffer_policy="maintain")
    s = _slowmo(w, guard=64)
    s.set_variant("outer", variant)
    s.set_variant("local", layout)
    s.run(2)
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()


@pytest.mark.parametrize("base,policy,m", [("nesterov", "average", 65), ("nesterov", "reset", 97), ("adam", "average", 66),
                                           ("adam", "reset", 129), ("adam", "maintain", 200)])
@pytest.mark.parametrize("variant", ["direct", "lazy"])
def test_derived_noise_keys_for_every_base_and_policy(base, policy, m, variant):
    # P chosen so that the last warp of the grid has lanes past the end of the row (they must stay in
    # the key-deriving loop without touching memory): 1030 columns = 258 groups = 8 warps + 2 lanes
    w = workloads.workload("tiny", P=1030, m=m, tau=3, T=2, base=base, buffer_policy=policy,
                           gamma=0.01 if base == "adam" else 0.05, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8, seed=8)
    s = _slowmo(w, guard=64)
    s.set_variant("outer", variant)
    s.run(2)
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()


def test_local_step_layouts_are_selectable_and_identical():
    import torch
    from paper_1910_00643_b200 import SlowMoError, binding
    outs = []
    for grad_mode in ("generated", "supplied"):
        for layout in ("row_tiles", "column_owner", "default"):
            w = workloads.workload("tiny", P=70_001, m=5, tau=3, T=2, grad_mode=grad_mode, buffer_policy="average")
            s = _slowmo(w)
            s.set_variant("local", layout)
            grad = None
            if grad_mode == "supplied":
                grad = s.alloc_gradient()
                s.fill_gradient()
            s.run(2, grad)
            _check_against_oracle(s, w, np.arange(0, w["P"], 7), exact=True)
            s.synchronize()
            outs.append(s.t["x"].view(w["m"], s.pitch)[:, :w["P"]].clone())   # padding columns are unspecified
            with pytest.raises(SlowMoError) as e:
                s.set_variant("local", "staged")        # an outer-step variant is not a local-step layout
            assert e.value.status == binding.EINVAL
            s.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    assert torch.equal(outs[3], outs[4]) and torch.equal(outs[3], outs[5])


def test_more_workers_than_one_grid_dimension_holds():
    # 66 000 rows: the creation-time fills stride over the rows, and every kernel derives its keys
    w = workloads.workload("tiny", P=9, m=66_000, tau=2, T=1, buffer_policy="average")
    s = _slowmo(w)
    s.run(1)
    ref = _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert ref["x"].shape == (66_000, 9)
    s.close()


def test_every_worker_holds_the_anchor_after_the_outer_step():
    import torch
    w = workloads.workload("tiny", P=10_001, m=6)
    s = _slowmo(w)
    s.run(2)
    s.synchronize()
    x = s.t["x"].view(6, s.pitch)[:, :w["P"]]
    assert bool((x == s.t["anchor"][:w["P"]].unsqueeze(0)).all())
    assert not bool(s.t["h"].view(6, s.pitch)[:, :w["P"]].any())  # reset policy
    s.close()


def test_runs_are_bit_reproducible():
    import torch
    w = workloads.workload("resnet50", P=200_003, m=8, T=2, n_tensors=0)
    outs = []
    for variant in ("direct", "staged", "direct", "fused", "lazy"):
        s = _slowmo(w)
        s.set_variant("outer", variant)
        s.run(2)
        s.materialize()      # raw tensors are read below; the lazy and fused variants defer some writes
        s.synchronize()
        outs.append([s.t[k].view(-1, s.pitch)[:, :w["P"]].clone() for k in ("x", "anchor", "u", "h")])
        s.close()
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert torch.equal(a, b)


def test_fused_last_step_is_transparent_through_the_api():
    # the deferred last inner step must be invisible: reading state between the inner loop and
    # the outer step runs it, and the run still ends bit-identical to the oracle
    w = workloads.workload("tiny", P=3000, m=3, tau=3, T=2, buffer_policy="maintain")
    ref_mid = oracle.run(oracle.make_config(**dict(w, T=1, alpha=1.0, beta=0.0)), j0=0, n=w["P"])
    s = _slowmo(w, guard=64)
    s.set_variant("outer", "fused")
    s.local_steps(3)
    h_mid = s.get_params("h")            # forces the deferred step; h after tau steps of iteration 0
    assert np.array_equal(h_mid.view(np.uint32), ref_mid["h"].view(np.uint32))
    s.outer_step()
    s.local_steps(2)
    s.local_steps(1)                     # deferred again, taken inside the outer-step kernel
    s.outer_step()
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()
    # tau = 1: every inner step is the last one
    w1 = workloads.workload("sync_sgd", P=2500, m=4, T=3)
    s = _slowmo(w1)
    s.set_variant("outer", "fused")
    s.run(3)
    _check_against_oracle(s, w1, np.arange(w1["P"]), exact=True)
    s.close()
    # supplied gradient
    w2 = workloads.workload("stress_tau12", P=4100, m=4, tau=2, T=2)
    s = _slowmo(w2)
    s.set_variant("outer", "fused")
    s.alloc_gradient()
    s.fill_gradient()
    s.run(2, s.grad)
    _check_against_oracle(s, w2, np.arange(w2["P"]), exact=True)
    s.close()


@pytest.mark.parametrize("base,policy", [("nesterov", "reset"), ("nesterov", "average"), ("nesterov", "maintain"),
                                         ("adam", "average"), ("adam", "reset")])
def test_lazy_broadcast_is_transparent_through_the_api(base, policy):
    import torch
    w = workloads.workload("tiny", P=3100, m=4, tau=3, T=3, base=base, buffer_policy=policy,
                           gamma=0.01 if base == "adam" else 0.05, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8)
    s = _slowmo(w, guard=64)
    s.set_variant("outer", "lazy")
    s.run(1)
    # the replicas are virtual now: the raw rows lag, the API does not
    ref1 = oracle.run(oracle.make_config(**dict(w, T=1)), j0=0, n=w["P"])
    assert np.array_equal(s.get_params("x").view(np.uint32), ref1["x"].view(np.uint32))   # materialises
    assert np.array_equal(s.get_params("h").view(np.uint32), ref1["h"].view(np.uint32))
    s.run(1)                                   # virtual again
    s.local_steps(1)                           # first step reads the anchor
    s.local_steps(2)
    s.outer_step()
    s.materialize()
    s.synchronize()
    x = s.t["x"].view(4, s.pitch)[:, :w["P"]]
    assert bool((x == s.t["anchor"][:w["P"]].unsqueeze(0)).all())     # raw tensors are up to date
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()
    # supplied gradient, and switching the variant while the replicas are virtual
    w2 = workloads.workload("stress_tau12", P=4100, m=3, tau=2, T=4)
    s = _slowmo(w2)
    s.set_variant("outer", "lazy")
    s.alloc_gradient()
    s.fill_gradient()
    s.run(2, s.grad)
    s.set_variant("outer", "staged")
    s.run(1, s.grad)
    s.set_variant("outer", "lazy")
    s.run(1, s.grad)
    _check_against_oracle(s, w2, np.arange(w2["P"]), exact=True)
    s.close()


def test_learning_rate_schedule():
    w = workloads.workload("tiny", P=2000, T=4)
    gammas = np.array([0.01, 0.05, 0.1, 0.02], np.float32)
    s = _slowmo(w)
    for t in range(4):
        s.set_gamma(float(gammas[t]))
        s.local_steps(w["tau"])
        s.outer_step()
    _check_against_oracle(s, w, np.arange(2000), gamma_t=gammas, exact=True)
    s.close()


def test_supplied_gradient_arrays_per_step():
    import torch
    m, tau, T, P = 3, 2, 2, 1500
    w = workloads.workload("stress_tau1", P=P, m=m, tau=tau, T=T, weight_decay=1e-2, buffer_policy="maintain")
    G = workloads.dense_gradients(T * tau, m, P, seed=9)
    s = _slowmo(w)
    g = s.alloc_gradient().view(m, s.pitch)
    step = 0
    for t in range(T):
        for k in range(tau):
            with torch.cuda.stream(s.stream):
                g[:, :P].copy_(torch.from_numpy(G[step]).cuda(), non_blocking=False)
            s.local_steps(1, s.grad)
            step += 1
        s.outer_step()
    cfg_w = dict(w, grad_mode="supplied_array")
    _check_against_oracle(s, cfg_w, np.arange(P), G=G, exact=True)
    s.close()


def test_supplied_hash_gradient_small():
    w = workloads.workload("stress_tau12", P=5000, m=4)
    s = _slowmo(w, guard=64)
    s.alloc_gradient()
    s.fill_gradient()
    s.run(w["T"], s.grad)
    _check_against_oracle(s, w, np.arange(5000), exact=True)
    assert s.guards_intact()
    s.close()


# ------------------------------------------------------------------ stochastic gradient push bases

@pytest.mark.parametrize("base,policy", [("sgp_nesterov", "reset"), ("sgp_nesterov", "average"),
                                         ("sgp_adam", "maintain"), ("sgp_adam", "reset")])
@pytest.mark.parametrize("m", [1, 2, 3, 8, 13, 32, 50, 64])
def test_sgp_small_runs_match_oracle(base, policy, m):
    w = workloads.workload("tiny", P=2 * 1024 + 37, m=m, tau=5, T=2, base=base, buffer_policy=policy, alpha=0.9,
                           beta=0.6, gamma=0.01 if "adam" in base else 0.05, weight_decay=1e-3, adam_b1=0.9,
                           adam_b2=0.98, adam_eps=1e-8, seed=9)
    s = _slowmo(w, guard=64)
    s.run(w["T"])
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()


def test_sgp_supplied_gradient_and_step_by_step_calls():
    w = workloads.workload("stress_tau12", P=3000, m=5, tau=7, T=2, base="sgp_nesterov")
    s = _slowmo(w)
    s.alloc_gradient()
    s.fill_gradient()
    for _ in range(2):
        for n in (3, 1, 3):        # the graph position must follow the global step count across calls
            s.local_steps(n, s.grad)
        s.outer_step()
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    s.close()


@pytest.mark.parametrize("base,policy", [("sgp_nesterov", "average"), ("sgp_adam", "reset"), ("sgp_nesterov", "maintain")])
@pytest.mark.parametrize("m", [65, 96, 128, 131])
def test_sgp_with_more_workers_than_inline_noise_keys(base, policy, m):
    # the walk along the cycles of i -> i + hops derives its keys 32 positions at a time; m = 96 and 131
    # give cycles whose length is not a multiple of 32, m = 128 several cycles per step
    w = workloads.workload("tiny", P=1030, m=m, tau=9, T=2, base=base, buffer_policy=policy, alpha=0.9, beta=0.6,
                           gamma=0.01 if "adam" in base else 0.05, weight_decay=1e-3, adam_b1=0.9, adam_b2=0.98,
                           adam_eps=1e-8, seed=10)
    s = _slowmo(w, guard=64)
    s.run(w["T"])
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()


@pytest.mark.parametrize("name", ["sgp_resnet50", "sgp_transformer_adam"])
def test_full_size_sgp_workloads_on_sampled_coordinates(name):
    import torch
    w = workloads.workload(name)
    s = _slowmo(w)
    s.run(w["T"])
    j = workloads.sample_coordinates(w["P"], 1 << 12, seed=3)
    _check_against_oracle(s, w, j, exact=True)
    x = s.t["x"].view(w["m"], s.pitch)[:, :w["P"]]
    assert bool((x == s.t["anchor"][:w["P"]].unsqueeze(0)).all())
    s.close()
    del s
    torch.cuda.empty_cache()


# ------------------------------------------------------- variant without the exact average (Section 6)

@pytest.mark.parametrize("base,policy", [("nesterov", "reset"), ("nesterov", "maintain"), ("adam", "maintain"),
                                         ("adam", "reset"), ("sgp_nesterov", "reset"), ("sgp_adam", "maintain")])
@pytest.mark.parametrize("m", [1, 3, 8])
def test_no_average_small_runs_match_oracle(base, policy, m):
    w = workloads.workload("tiny", P=2 * 1024 + 37, m=m, tau=4, T=3, base=base, buffer_policy=policy, alpha=0.9,
                           beta=0.6, gamma=0.01 if "adam" in base else 0.05, weight_decay=1e-3, adam_b1=0.9,
                           adam_b2=0.98, adam_eps=1e-8, seed=12, no_average=True)
    s = _slowmo(w, guard=64)
    s.set_variant("outer", "fused")      # has no effect without the average
    s.run(w["T"])
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.get_params("anchor").shape == (m, w["P"]) and s.get_params("u", replica=m - 1).shape == (1, w["P"])
    assert s.guards_intact()
    s.close()


def test_no_average_refuses_the_average_policy():
    from paper_1910_00643_b200 import SlowMoError, binding
    with pytest.raises(SlowMoError) as e:
        _slowmo(workloads.workload("tiny", buffer_policy="average", no_average=True))
    assert e.value.status == binding.EINVAL


def test_full_size_sgp_without_the_average_on_sampled_coordinates():
    import torch
    w = workloads.workload("sgp_resnet50", T=2, no_average=True)
    s = _slowmo(w)
    s.run(w["T"])
    j = workloads.sample_coordinates(w["P"], 1 << 12, seed=4)
    _check_against_oracle(s, w, j, exact=True)
    x = s.t["x"].view(w["m"], s.pitch)[:, :w["P"]]
    anchor = s.t["anchor"].view(w["m"], s.pitch)[:, :w["P"]]
    assert torch.equal(x, anchor)                       # each worker restarts from its own outer iterate
    assert not bool((x == x[0:1]).all())                # and the workers no longer agree
    s.close()
    del s
    torch.cuda.empty_cache()


# --------------------------------------------------------------------------- boundary behaviour

def test_call_order_and_argument_errors():
    from paper_1910_00643_b200 import SlowMoError, binding
    import torch
    w = workloads.workload("tiny")
    s = _slowmo(w)
    with pytest.raises(SlowMoError) as e:
        s.outer_step()                       # no local steps yet
    assert e.value.status == binding.ESTATE
    s.local_steps(3)
    with pytest.raises(SlowMoError) as e:
        s.local_steps(2)                     # 3 + 2 > tau
    assert e.value.status == binding.ESTATE
    with pytest.raises(SlowMoError) as e:
        s.set_gamma(0.1)                     # only legal at k = 0
    assert e.value.status == binding.ESTATE
    with pytest.raises(SlowMoError) as e:
        s.local_steps(1, torch.zeros(4 * s.pitch, device="cuda"))  # gradient given in generated mode
    assert e.value.status == binding.EINVAL
    s.local_steps(1)
    s.outer_step()
    with pytest.raises(SlowMoError) as e:
        s.set_gamma(float("nan"))
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        s.get_params("x", replica=4)
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        s.get_params("anchor", offset=4000, count=200)
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        s.get_params("v")                    # Nesterov has no second moment
    assert e.value.status == binding.EINVAL
    assert s.counters() == (1, 0, 0)
    s.sync_status()
    s.close()
    ws = workloads.workload("stress_tau1", P=1000)
    s = _slowmo(ws)
    with pytest.raises(SlowMoError) as e:
        s.local_steps(1)                     # supplied mode needs a gradient
    assert e.value.status == binding.EINVAL
    s.close()


def test_empty_requests_are_accepted_and_change_nothing():
    # zero inner steps, zero columns, zero noise draws: legal no-ops at any point of the loop
    import torch
    w = workloads.workload("tiny", P=37, m=3)
    s = _slowmo(w, guard=64)
    s.local_steps(2)
    before = {k: s.get_params(k).copy() for k in _state_keys(w)}
    s.local_steps(0)
    assert s.counters() == (0, 2, 2)
    assert s.get_params("x", offset=37, count=0).shape == (3, 0)
    assert s.get_params("anchor", offset=5, count=0).shape == (1, 0)
    s.set_params("u", np.zeros(1, np.float32), offset=0, count=0)
    s.debug_noise(3, 0, 0, 0, 0, 0)
    for k in _state_keys(w):
        assert np.array_equal(before[k].view(np.uint32), s.get_params(k).view(np.uint32)), k
    s.local_steps(w["tau"] - 2)
    s.outer_step()
    s.run(w["T"] - 1)
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    assert s.guards_intact()
    s.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_survives():
    from paper_1910_00643_b200 import SlowMoError, binding
    w = workloads.workload("tiny", P=3000)
    s = _slowmo(w)
    s.set_variant("outer", "staged")
    s.run(1)
    s.sync_status()                       # clean so far
    s.debug_wait_timeout(4096)            # a wait on a barrier nothing completes
    with pytest.raises(SlowMoError) as e:
        s.sync_status()
    assert e.value.status == binding.ETIMEOUT
    s.sync_status()                       # the record is cleared, the context still works
    s.run(2)
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    s.close()


@pytest.mark.parametrize("name,over,variant,chunks", [
    ("tiny", dict(P=10_007, m=3, tau=3, buffer_policy="average"), "fused", 3),
    ("tiny", dict(P=10_007, m=3, tau=3, buffer_policy="reset"), "staged", 4),
    ("transformer_adam", dict(P=9_001, m=4, tau=2), "direct", 2),
    ("sgp_resnet50", dict(P=12_345, m=5, tau=4), "direct", 5),
    ("tiny", dict(P=7_000, m=3, tau=2, buffer_policy="maintain", no_average=True), "direct", 3),
    ("tiny", dict(P=100, m=2, tau=1), "fused", 8),
    ("tiny", dict(P=10_007, m=3, tau=3, buffer_policy="average"), "lazy", 3),
    ("transformer_adam", dict(P=9_001, m=4, tau=2, buffer_policy="reset"), "lazy", 2),
])
def test_pipelined_host_iteration_equals_the_plain_call_sequence(name, over, variant, chunks):
    import torch
    w = workloads.workload(name, **over)
    P, m = w["P"], w["m"]
    rng = np.random.Generator(np.random.PCG64(5))
    a, b = _slowmo(w, guard=64), _slowmo(w, guard=64)
    for s in (a, b):
        s.set_variant("outer", variant)
    rows = m if w.get("no_average") else 1
    for it in range(3):
        c_host = torch.from_numpy(rng.standard_normal((m, P)).astype(np.float32)).pin_memory()
        out_host = torch.empty((rows, P), dtype=torch.float32).pin_memory()
        a.iteration_host(c_host, out_host, chunks)          # pipelined
        b.set_params("c", c_host)                            # plain sequence
        b.local_steps(w["tau"])
        b.outer_step()
        ref = b.get_params("anchor")
        assert np.array_equal(out_host.numpy().view(np.uint32), ref.view(np.uint32)), it
    for key in _state_keys(w):
        assert np.array_equal(a.get_params(key).view(np.uint32), b.get_params(key).view(np.uint32)), key
    assert a.counters() == b.counters()
    assert a.guards_intact() and b.guards_intact()
    a.close()
    b.close()


def test_get_and_set_params_round_trip():
    import torch
    w = workloads.workload("tiny", P=3001, m=3)
    s = _slowmo(w, guard=64)
    s.run(1)
    x = s.get_params("x")
    assert x.shape == (3, 3001)
    row1 = s.get_params("x", replica=1, offset=100, count=50)
    assert np.array_equal(row1[0], x[1, 100:150])
    dev = torch.empty(3 * 40, dtype=torch.float32, device="cuda")
    s.get_params("h", offset=7, count=40, out=dev)
    s.synchronize()
    assert np.array_equal(dev.cpu().numpy().reshape(3, 40), s.get_params("h")[:, 7:47])
    # restore a checkpoint into a fresh context and continue: same result as an uninterrupted run
    s2 = _slowmo(w)
    s2.set_state(**s.get_state())
    for key in ("x", "anchor", "u", "h"):
        s2.set_params(key, s.get_params(key))
    s.run(2)
    s2.run(2)
    for key in ("x", "anchor", "u", "h"):
        assert np.array_equal(s2.get_params(key).view(np.uint32), s.get_params(key).view(np.uint32)), key
    _check_against_oracle(s2, w, np.arange(w["P"]), T=3, exact=True)
    assert s.guards_intact()
    s.close()
    s2.close()


def _checkpoint(s):
    """Everything Algorithm 1 carries, on the host: the tensors and the position record."""
    keys = ("x", "anchor", "u", "h") + (("v",) if s.t["v"] is not None else ())
    return {"state": s.get_state(), "tensors": {k: s.get_params(k) for k in keys}}


def _restore(s, ck):
    s.set_state(**ck["state"])
    for k, v in ck["tensors"].items():
        s.set_params(k, np.ascontiguousarray(v))


CHECKPOINT_CASES = {
    "nesterov-generated-reset": dict(base="nesterov", buffer_policy="reset"),
    "nesterov-generated-average": dict(base="nesterov", buffer_policy="average", weight_decay=1e-3),
    "adam-maintain": dict(base="adam", buffer_policy="maintain", gamma=0.01, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8),
    "adam-reset": dict(base="adam", buffer_policy="reset", gamma=0.01, adam_b1=0.9, adam_b2=0.98, adam_eps=1e-8),
    "sgp-nesterov-maintain": dict(base="sgp_nesterov", buffer_policy="maintain", m=6),
    "sgp-adam-average": dict(base="sgp_adam", buffer_policy="average", gamma=0.01, adam_b1=0.9, adam_b2=0.98,
                             adam_eps=1e-8, m=5),
    "noaverage-adam": dict(base="adam", buffer_policy="maintain", gamma=0.01, adam_b1=0.9, adam_b2=0.98,
                           adam_eps=1e-8, no_average=True),
}


@pytest.mark.parametrize("variant", ["direct", "lazy"])
@pytest.mark.parametrize("k_split", [0, 2, 5])       # restore between outer iterations, inside one, and with the outer step due
@pytest.mark.parametrize("case", sorted(CHECKPOINT_CASES))
def test_a_restored_run_continues_bit_identically(case, k_split, variant):
    # T1 iterations (+ k_split inner steps), checkpoint, fresh context, restore, the rest: the result
    # must equal the uninterrupted run and the oracle bit for bit, with a changing gamma_t
    T1, T2, tau = 2, 2, 5
    w = workloads.workload("tiny", **dict(dict(P=2 * 1024 + 37, m=4, tau=tau, T=T1 + T2, alpha=0.9, beta=0.6, seed=14),
                                          **CHECKPOINT_CASES[case]))
    gammas = (w["gamma"] * np.array([1.0, 0.5, 2.0, 0.7])).astype(np.float32)

    def advance(s, t_from, t_to, k_from=0):
        for t in range(t_from, t_to):
            if k_from == 0:
                s.set_gamma(float(gammas[t]))
            if tau - k_from:
                s.local_steps(tau - k_from)
            s.outer_step()
            k_from = 0

    first = _slowmo(w, guard=64)
    first.set_variant("outer", variant)
    advance(first, 0, T1)
    if k_split:
        first.set_gamma(float(gammas[T1]))
        first.local_steps(k_split)
    ck = _checkpoint(first)
    assert ck["state"]["t"] == T1 and ck["state"]["k"] == k_split
    assert ck["state"]["gamma_t"] == (gammas[T1] if k_split else gammas[T1 - 1])
    first.close()

    second = _slowmo(w, guard=64)
    second.set_variant("outer", variant)
    _restore(second, ck)
    assert second.counters() == (T1, k_split, ck["state"]["l"])
    advance(second, T1, T1 + T2, k_from=k_split)
    _check_against_oracle(second, w, np.arange(w["P"]), gamma_t=gammas, exact=True)
    assert second.guards_intact()
    second.close()


def test_set_state_refuses_impossible_positions_and_flushes_what_is_owed():
    from paper_1910_00643_b200 import SlowMoError, binding
    w = workloads.workload("tiny", P=3000, m=3, tau=3, T=2)
    s = _slowmo(w)
    for bad in (dict(t=0, k=4, l=4, gamma_t=0.05),            # k > tau
                dict(t=0, k=1, l=0, gamma_t=0.05),            # fewer steps since the reset than steps in this iteration
                dict(t=3, k=1, l=7, gamma_t=0.05),            # reset policy: l must equal k
                dict(t=0, k=0, l=0, gamma_t=0.0), dict(t=0, k=0, l=0, gamma_t=float("nan"))):
        with pytest.raises(SlowMoError) as e:
            s.set_state(**bad)
        assert e.value.status == binding.EINVAL
    # a lazy context owes its tensors the broadcast: set_state writes it out before moving on
    s.set_variant("outer", "lazy")
    s.run(1)
    ref = oracle.run(oracle.make_config(**dict(w, T=1)), j0=0, n=w["P"])
    s.set_state(t=1, k=0, l=0, gamma_t=w["gamma"])
    s.synchronize()
    x = s.t["x"].view(3, s.pitch)[:, :w["P"]].cpu().numpy()
    assert np.array_equal(x.view(np.uint32), ref["x"].view(np.uint32))
    s.run(1)
    _check_against_oracle(s, w, np.arange(w["P"]), exact=True)
    # with the buffers kept, l keeps counting across outer iterations: a large count is legal and
    # its powers underflow to zero without harm
    wm = workloads.workload("tiny", P=100, m=2, tau=3, base="adam", buffer_policy="maintain", gamma=0.01)
    sm = _slowmo(wm)
    sm.set_state(t=10**6, k=0, l=3 * 10**6, gamma_t=0.01)
    sm.run(1)
    assert sm.get_state() == {"t": 10**6 + 1, "k": 0, "l": 3 * 10**6 + 3, "gamma_t": np.float32(0.01)}
    sm.close()
    s.close()


def test_tensor_table():
    w = workloads.workload("resnet50", P=100_000, m=2, T=1, tau=1)
    s = _slowmo(w)
    sizes = workloads.tensor_sizes(100_000, 161, 0)
    assert int(sizes.sum()) == 100_000 and sizes.min() >= 1
    off = 0
    for i in (0, 1, 80, 160):
        o, c = s.tensor_range(i)
        assert o == int(sizes[:i].sum()) and c == int(sizes[i])
    from paper_1910_00643_b200 import SlowMoError
    with pytest.raises(SlowMoError):
        s.tensor_range(161)
    s.close()


# ------------------------------------------------------- full benchmark sizes
#
# Each full-size run is compared with the oracle on (i) sampled coordinates (both ends, tile
# boundaries, 8192 uniform draws) and (ii) three contiguous slabs of 2^20 coordinates: the start of
# the vector, the middle, and the end with its ragged tail (for the 1e9-parameter workload the middle
# slab straddles the point where row 1's byte offset passes 2^32). Properties that hold at any size
# (every replica equals the anchor, policy post-conditions) are checked over the whole of P. The
# fraction of P compared element by element is asserted below; `-m fullp` runs compare all of it.

FULL = ["resnet50", "bmuf", "local_sgd", "sync_sgd", "transformer_adam"]
SLAB = 1 << 20


def _slabs(w, pitch):
    P = w["P"]
    mid = (P // 2 // 4096) * 4096 - SLAB // 2 + 13         # unaligned start, crosses tile boundaries
    if P * 4 > 2**32:                                      # rows longer than 4 GiB apart: straddle row 1's 2^32-byte mark
        mid = (2**32 - pitch * 4) // 4 - SLAB // 2
    return [np.arange(0, SLAB), np.arange(mid, mid + SLAB), np.arange(P - SLAB, P)]


def _check_full_size(s, w, seed, slabs=True, gamma_t=None):
    import torch
    j = workloads.sample_coordinates(w["P"], 1 << 13, seed=seed)
    _check_against_oracle(s, w, j, exact=True, gamma_t=gamma_t)
    compared = len(j)
    if slabs:
        for slab in _slabs(w, s.pitch):
            _check_against_oracle(s, w, slab, exact=True, gamma_t=gamma_t)
            compared += len(slab)
        assert compared >= 3 * SLAB
    if not w.get("no_average"):
        x = s.t["x"].view(w["m"], s.pitch)[:, :w["P"]]
        assert bool((x == s.t["anchor"][:w["P"]].unsqueeze(0)).all())     # consensus over the whole of P
    h = s.t["h"].view(w["m"], s.pitch)[:, :w["P"]]
    if w["buffer_policy"] == "reset":
        assert not bool(h.any())
    if w["buffer_policy"] == "average":
        assert bool((h == h[0:1]).all())
    assert bool(torch.isfinite(s.t["u"].view(-1, s.pitch)[:, :w["P"]]).all())
    return compared


def _free(s):
    import torch
    s.close()
    del s
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", FULL)
def test_full_size_generated_workloads(name):
    w = workloads.workload(name)
    s = _slowmo(w)
    s.run(w["T"])
    # slabs for the three workloads that differ in kernel and policy (resnet50: Nesterov / average,
    # bmuf: reset, transformer_adam: Adam / maintain); the two degenerate cases share bmuf's kernels
    _check_full_size(s, w, seed=1, slabs=name in ("resnet50", "bmuf", "transformer_adam"))
    _free(s)


@pytest.mark.parametrize("name,variant", [("stress_tau1", "direct"), ("stress_tau12", "direct"),
                                          ("stress_tau12", "lazy"), ("stress_tau1", "fused"),
                                          ("stress_tau48", "direct"), ("stress_tau48", "lazy"),
                                          ("stress_tau12", "staged")])
def test_full_size_supplied_gradient(name, variant):
    w = workloads.workload(name)
    s = _slowmo(w)
    s.set_variant("outer", variant)
    s.alloc_gradient()
    s.fill_gradient()
    s.run(w["T"], s.grad)
    _check_full_size(s, w, seed=2)       # reads through sync_status, which writes out lazy state
    _free(s)


@pytest.mark.parametrize("name,variant,layout", [("bmuf", "staged", "default"), ("bmuf", "lazy", "default"),
                                                 ("resnet50", "lazy", "default"), ("resnet50", "staged", "row_tiles"),
                                                 ("transformer_adam", "lazy", "row_tiles")])
def test_full_size_other_variants_and_layouts(name, variant, layout):
    # the staged (bulk-copy) outer step on a reset policy, the lazy variant at every policy, and the
    # row-tile layout of the generated-gradient local step, each at full size (two outer iterations)
    w = workloads.workload(name, T=2)
    s = _slowmo(w)
    s.set_variant("outer", variant)
    s.set_variant("local", layout)
    s.run(2)
    _check_full_size(s, w, seed=5, slabs=False)
    _check_against_oracle(s, w, _slabs(w, s.pitch)[1][:1 << 18], exact=True)
    _free(s)


@pytest.mark.parametrize("layout", ["row_tiles", "column_owner"])
def test_full_size_with_more_workers_than_inline_noise_keys(layout):
    # m = 70 > 64: the kernels derive the row keys themselves; P = 2^24 + 5 (ragged), 4.7 GB of state
    w = workloads.workload("resnet50", P=(1 << 24) + 5, m=70, tau=4, T=2, n_tensors=0)
    s = _slowmo(w)
    s.set_variant("local", layout)
    s.set_variant("outer", "lazy" if layout == "column_owner" else "direct")
    s.run(2)
    _check_full_size(s, w, seed=6, slabs=False)
    _check_against_oracle(s, w, np.arange(w["P"] - (1 << 17), w["P"]), exact=True)
    _free(s)


@pytest.mark.parametrize("P,grad_mode,m,variant,layout", [
    (2**32 - 4096, "generated", 1, "direct", "column_owner"), (2**32 - 4096, "supplied", 2, "lazy", "default"),
    (2**32 + 2**20 + 5, "generated", 1, "direct", "column_owner"), (2**32 + 2**20 + 5, "generated", 1, "staged", "row_tiles"),
    (2**32 + 2**20 + 5, "supplied", 2, "lazy", "default"), (2**32 + 2**20 + 5, "supplied", 2, "fused", "default"),
    (6_400_000_003, "supplied", 1, "direct", "row_tiles"), (6_400_000_003, "supplied", 1, "staged", "column_owner")])
def test_parameter_counts_around_and_beyond_two_to_the_32(P, grad_mode, m, variant, layout):
    # Rows of 17 to 26 GB (100-145 GB of state): column offsets pass 2^32 inside a row, so every kernel's
    # index arithmetic beyond 32 bits is exercised. (The library's own limit, SLOWMO_MAX_P = 2^34 - 16384,
    # is more than one B200 holds; its refusal is a host test.) Compared with the oracle at both ends,
    # around the columns 2^30, 2^31 and 2^32, in the last tiles, and on sampled coordinates.
    import gc
    import torch
    gc.collect()
    torch.cuda.empty_cache()          # memory cached from earlier tests counts as free
    free, _ = torch.cuda.mem_get_info()
    need = 4 * P * ((3 * m + 3) if grad_mode == "generated" else (3 * m + 2)) + (8 << 30)
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free")
    w = workloads.workload("resnet50", P=P, m=m, tau=2, T=2, n_tensors=0, grad_mode=grad_mode, sigma=0.05)
    s = _slowmo(w)
    s.set_variant("outer", variant)
    s.set_variant("local", layout)
    grad = None
    if grad_mode == "supplied":
        grad = s.alloc_gradient()
        s.fill_gradient()
    s.run(2, grad)
    _check_full_size(s, w, seed=9, slabs=False)
    near = [np.arange(0, 1 << 16), np.arange(P - (1 << 16), P)]
    near += [np.arange(b - 4100, b + 4100) for b in (2**30, 2**31, 2**32) if b + 4100 < P]
    _check_against_oracle(s, w, np.concatenate(near), exact=True)
    _free(s)


def test_full_size_staged_and_fused_outer_steps_equal_direct():
    import torch
    w = workloads.workload("resnet50", T=2)
    res = []
    for variant in ("direct", "staged", "fused", "lazy"):
        s = _slowmo(w)
        s.set_variant("outer", variant)
        s.run(2)
        s.sync_status()
        res.append((s.t["anchor"].clone(), s.t["u"].clone(), s.t["h"].view(w["m"], s.pitch)[::8].clone(),
                    s.t["x"].view(w["m"], s.pitch)[::8].clone()))
        _free(s)
    for other in res[1:]:
        for a, b in zip(res[0], other):
            assert torch.equal(a[..., :w["P"]], b[..., :w["P"]])


# ------------------------------------------------------- every coordinate of a full-size workload

FULLP_CHUNK = 1 << 22


@pytest.mark.fullp
@pytest.mark.parametrize("name,variants", [
    ("resnet50", ("direct", "staged", "fused", "lazy")), ("bmuf", ("direct", "staged", "lazy")),
    ("local_sgd", ("direct", "lazy")), ("sync_sgd", ("direct", "fused")),
    ("transformer_adam", ("direct", "fused", "lazy")),
    ("sgp_resnet50", ("direct",)), ("sgp_transformer_adam", ("direct",)),
    ("stress_tau1", ("direct", "fused")), ("stress_tau12", ("direct", "lazy")), ("stress_tau48", ("direct", "lazy"))])
def test_every_coordinate_of_a_full_size_workload(name, variants):
    """Selected with -m fullp only (minutes of oracle time per workload). Every named variant runs the
    whole workload on the GPU; then the oracle goes over the vector once, in chunks of 2^22 coordinates,
    and every element of every state tensor of every variant is compared with it bit for bit. The count
    of coordinates compared and of unequal elements is printed (run with -s) and, when the environment
    variable SLOWMO_FULLP_OUT names a folder, written to fullp_<name>.txt there."""
    import os
    import time
    w = workloads.workload(name)
    runs = []
    for variant in variants:
        s = _slowmo(w)
        s.set_variant("outer", variant)
        grad = None
        if w["grad_mode"] == "supplied":
            grad = s.alloc_gradient()
            s.fill_gradient()
        s.run(w["T"], grad)
        s.sync_status()
        runs.append(s)
    cfg = oracle.make_config(**w)
    unequal, compared, t0 = [0] * len(runs), 0, time.time()
    for j0 in range(0, w["P"], FULLP_CHUNK):
        n = min(FULLP_CHUNK, w["P"] - j0)
        ref = oracle.run(cfg, j0=j0, n=n, precision="f32")
        for i, s in enumerate(runs):
            for key in _state_keys(w):
                got = s.get_params(key, offset=j0, count=n).reshape(ref[key].shape)
                unequal[i] += int((got.view(np.uint32) != ref[key].view(np.uint32)).sum())
        compared += n
    lines = [f"{name} ({variant}): {compared} of {w['P']} coordinates compared, all m={w['m']} workers, "
             f"tensors {','.join(_state_keys(w))}: {bad} unequal elements"
             for variant, bad in zip(variants, unequal)]
    lines.append(f"{name}: {time.time() - t0:.0f} s")
    print("\n".join(lines))
    out = os.environ.get("SLOWMO_FULLP_OUT", "")
    if out and os.path.isdir(out):
        with open(os.path.join(out, f"fullp_{name}.txt"), "w") as f:
            f.write("\n".join(lines) + "\n")
    assert compared == w["P"] and not any(unequal), lines
    for s in runs:
        _free(s)


# ------------------------------------------------------------------ seeded random configurations

def _random_case(rng):
    base = rng.choice(["nesterov", "adam", "sgp_nesterov", "sgp_adam"])
    no_average = bool(rng.random() < 0.25)
    policy = rng.choice(["reset", "maintain"] if no_average else ["reset", "maintain", "average"])
    supplied = bool(rng.random() < 0.3)
    m = int(rng.choice([1, 2, 3, 5, 7, 8, 16, 33, 64]))
    return dict(P=int(rng.integers(1, 6000)), m=m, tau=int(rng.integers(1, 6)), T=int(rng.integers(1, 4)),
                alpha=float(rng.choice([1.0, 0.5, 1.5])), beta=float(rng.choice([0.0, 0.5, 0.9])),
                gamma=float(rng.choice([1e-3, 0.01])) if "adam" in base else float(rng.choice([0.01, 0.1])),
                base=str(base), mu=float(rng.choice([0.0, 0.9])), weight_decay=float(rng.choice([0.0, 1e-4, 1e-2])),
                adam_b1=0.9, adam_b2=float(rng.choice([0.98, 0.999])), adam_eps=float(rng.choice([1e-8, 1e-6])),
                buffer_policy=str(policy), grad_mode="supplied" if supplied else "generated",
                seed=int(rng.integers(0, 2**40)), a_lo=0.1, a_hi=float(rng.choice([1.0, 3.0])),
                c_std=float(rng.choice([0.05, 1.0])), sigma=float(rng.choice([0.0, 0.01, 0.3])),
                x_init=float(rng.choice([0.0, -0.5])), no_average=no_average)


@pytest.mark.parametrize("case", range(72))
def test_seeded_random_configurations_match_the_oracle(case):
    rng = np.random.Generator(np.random.PCG64(1000 + case))
    w = _random_case(rng)
    variant = str(rng.choice(["direct", "staged", "fused", "lazy"]))
    layout = "default"
    if case >= 48:   # more workers than noise keys fit the kernel arguments, either local-step layout
        w.update(m=int(rng.choice([65, 96, 130])), P=int(rng.integers(1, 1500)))
        layout = str(rng.choice(["default", "row_tiles", "column_owner"]))
    s = _slowmo(w, guard=64)
    s.set_variant("outer", variant)
    s.set_variant("local", layout)
    grad = None
    if w["grad_mode"] == "supplied":
        grad = s.alloc_gradient()
        s.fill_gradient()
    gammas = None
    if rng.random() < 0.3:   # a changing base learning rate
        gammas = (w["gamma"] * rng.uniform(0.5, 2.0, size=w["T"])).astype(np.float32)
    for t in range(w["T"]):
        if gammas is not None:
            s.set_gamma(float(gammas[t]))
        left = w["tau"]
        while left:          # the inner loop in random pieces
            n = int(rng.integers(1, left + 1))
            s.local_steps(n, grad)
            left -= n
        s.outer_step()
    _check_against_oracle(s, w, np.arange(w["P"]), gamma_t=gammas, exact=True)
    assert s.guards_intact(), (w, variant)
    s.close()
