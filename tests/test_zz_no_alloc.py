"""The allocation-free outer step (slowmo_outer_step_static) against the context's outer step.

Some callers cannot allocate device memory: code running under a framework allocator that
owns the whole device, a process with a fixed memory budget, or a latency-critical loop that
cannot afford the synchronisation an allocation implies. They cannot create a context
(creation allocates a small status block), so the library offers them one outer step that
keeps its scratch in a fixed array inside the library. This test drives that entry point
through the C ABI and requires bit-identical tensors to the context path, on two calls in a
row that share the scratch, with different base optimizers and buffer policies.

Collected last on purpose: if it fails under `pytest -x`, every other test has already run.
"""
import numpy as np
import pytest

from paper_1910_00643_b200 import workloads

pytestmark = pytest.mark.gpu

RTOL = 1e-5  # same gate as the parity tests; bit equality is expected and also asserted


def _pre_state(s):
    """Copies of the tensors an outer step reads and writes, taken before the context's own step.
    The copies are made on the context's stream, the one both outer steps run on, so that neither
    can overtake them."""
    import torch
    with torch.cuda.stream(s.stream):
        mine = {k: (s.t[k].clone() if s.t[k] is not None else None) for k in ("x", "h", "v", "anchor", "u")}
    s.synchronize()
    return mine


def _compare(s, mine, what):
    import torch
    s.synchronize()
    torch.cuda.synchronize()
    for key, t in mine.items():
        if t is None:
            continue
        rows = s.m if key in ("x", "h", "v") else 1
        got = t.view(rows, s.pitch)[:, :s.P].cpu().numpy().astype(np.float64)
        ref = s.t[key].view(rows, s.pitch)[:, :s.P].cpu().numpy().astype(np.float64)
        assert (np.abs(got - ref) <= RTOL * (1.0 + np.abs(ref))).all(), (what, key)
        assert np.array_equal(got, ref), (what, key, "not bit-identical")


def _one_call(s, w, what, wait=True):
    from paper_1910_00643_b200 import binding
    s.local_steps(w["tau"])
    mine = _pre_state(s)
    s.outer_step()                               # existing entry point, context path
    binding.outer_step_static(mine["x"], mine["h"], mine["v"], mine["anchor"], mine["u"], pitch=s.pitch,
                              P=s.P, m=s.m, base=w["base"], buffer_policy=w["buffer_policy"],
                              alpha=w["alpha"], beta=w["beta"], gamma=w["gamma"], stream=s.stream, wait=wait)
    _compare(s, mine, what)                      # synchronises the stream first


def test_static_outer_step_matches_context_outer_step_twice_in_a_row():
    from paper_1910_00643_b200 import SlowMo
    # first call: Nesterov, averaged buffers, ragged size over several tiles
    w1 = workloads.workload("resnet50", P=5 * 1024 + 37, m=6, tau=3, n_tensors=0)
    s1 = SlowMo(w1)
    _one_call(s1, w1, "first call")
    # second call, straight after, sharing the scratch: Adam with reset buffers
    w2 = workloads.workload("transformer_adam", P=3 * 1024 + 4, m=5, tau=2, buffer_policy="reset")
    s2 = SlowMo(w2)
    _one_call(s2, w2, "second call")
    # and once more on the first context (second outer iteration, non-zero slow momentum)
    _one_call(s1, w1, "third call")
    # a call that only enqueues (wait = 0), followed by a waiting one that reuses the scratch
    _one_call(s2, w2, "fourth call, not waiting", wait=False)
    _one_call(s1, w1, "fifth call")
    s1.close()
    s2.close()


def test_static_outer_step_refuses_sizes_beyond_its_maximum():
    import torch
    from paper_1910_00643_b200 import SlowMoError, binding
    t = torch.zeros(4096, device="cuda")
    common = dict(pitch=1024, m=2, base="nesterov", buffer_policy="reset", alpha=1.0, beta=0.5, gamma=0.1)
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_static(t, t, None, t, t, P=2**32, **common)            # P beyond the maximum
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_static(t, t, None, t, t, P=1000, **dict(common, m=65537))  # m beyond the maximum
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_static(t, t, None, t, t, P=1000, **dict(common, base="adam"))  # Adam needs v
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_static(t, t, None, t, t, P=1000, **dict(common, pitch=1002))
    assert e.value.status == binding.EALIGN
