"""Worker-sharded outer step (slowmo_outer_step_sharded): several GPUs' worth of state, emulated
on one GPU as separate buffer sets whose pointers stand for the peer mappings. The per-GPU kernels
never wait on one another, so running them one after the other on one device is the same
computation. The result must be bit-identical to one context holding all workers, and to the
oracle."""
import numpy as np
import pytest

import oracle
from paper_1910_00643_b200 import workloads

pytestmark = pytest.mark.gpu


def _run_sharded(w, world, T):
    """`world` contexts with m/world workers each (worker_offset set), local steps per context,
    one sharded outer-step call per emulated GPU. Returns the contexts."""
    import torch
    from paper_1910_00643_b200 import SlowMo, binding
    m_local = w["m"] // world
    stream = torch.cuda.Stream()
    ranks = [SlowMo(dict(w, m=m_local, worker_offset=r * m_local), stream=stream, guard=64) for r in range(world)]
    adam = "adam" in w["base"]
    for _ in range(T):
        for s in ranks:
            s.local_steps(w["tau"])
        # (on real GPUs: a stream-ordered collective here, so every GPU's rows are final)
        for r in range(world):
            binding.outer_step_sharded(
                r, [s.t["x"] for s in ranks], [s.t["h"] for s in ranks], [s.t["v"] for s in ranks] if adam else None,
                [s.t["anchor"] for s in ranks], [s.t["u"] for s in ranks], m_local=m_local, P=w["P"], pitch=ranks[0].pitch,
                base=w["base"], buffer_policy=w["buffer_policy"], alpha=w["alpha"], beta=w["beta"], gamma=w["gamma"],
                stream=stream)
        # (and here, before anyone's next local step)
        for s in ranks:
            s.outer_step_external()
    return ranks


@pytest.mark.parametrize("base,policy", [("nesterov", "reset"), ("nesterov", "average"), ("nesterov", "maintain"),
                                         ("adam", "maintain"), ("adam", "average")])
@pytest.mark.parametrize("world,m", [(1, 3), (2, 4), (4, 8), (3, 6), (8, 8)])
def test_sharded_outer_step_matches_one_context_and_the_oracle(base, policy, world, m):
    P = 4 * 1024 + 37
    w = workloads.workload("tiny", P=P, m=m, tau=3, T=3, base=base, buffer_policy=policy, alpha=0.9, beta=0.6,
                           gamma=0.01 if base == "adam" else 0.05, weight_decay=1e-3, adam_b1=0.9, adam_b2=0.98,
                           adam_eps=1e-8, seed=21)
    ranks = _run_sharded(w, world, w["T"])
    ref = oracle.run(oracle.make_config(**w), j0=0, n=P, precision="f32")
    m_local = m // world
    keys = ("x", "h") + (("v",) if base == "adam" else ())
    for r, s in enumerate(ranks):
        for key in keys:
            got = s.get_params(key)
            want = ref[key][r * m_local:(r + 1) * m_local]
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (r, key)
        # every GPU holds the same full copy of the outer iterate and of the slow momentum
        assert np.array_equal(s.get_params("anchor")[0].view(np.uint32), ref["anchor"].view(np.uint32)), r
        assert np.array_equal(s.get_params("u")[0].view(np.uint32), ref["u"].view(np.uint32)), r
        assert s.counters()[:2] == (3, 0)
        assert s.guards_intact()
        s.close()


def test_sharded_outer_step_with_a_deferred_last_step_and_bad_arguments():
    import torch
    from paper_1910_00643_b200 import SlowMo, SlowMoError, binding
    w = workloads.workload("tiny", P=3001, m=4, tau=2, T=2, buffer_policy="average")
    # the fused variant defers the last local step; slowmo_outer_step_external must not lose it
    m_local, world = 2, 2
    stream = torch.cuda.Stream()
    ranks = [SlowMo(dict(w, m=m_local, worker_offset=r * m_local), stream=stream) for r in range(world)]
    for s in ranks:
        s.set_variant("outer", "fused")
    for _ in range(2):
        for s in ranks:
            s.local_steps(2)
            s.materialize()          # rows must be final before peers read them
        for r in range(world):
            binding.outer_step_sharded(r, [s.t["x"] for s in ranks], [s.t["h"] for s in ranks], None,
                                       [s.t["anchor"] for s in ranks], [s.t["u"] for s in ranks], m_local=m_local,
                                       P=w["P"], pitch=ranks[0].pitch, base="nesterov", buffer_policy="average",
                                       alpha=w["alpha"], beta=w["beta"], gamma=w["gamma"], stream=stream)
        for s in ranks:
            s.outer_step_external()
    ref = oracle.run(oracle.make_config(**w), j0=0, n=w["P"], precision="f32")
    for r, s in enumerate(ranks):
        assert np.array_equal(s.get_params("x").view(np.uint32), ref["x"][2 * r:2 * r + 2].view(np.uint32))
    s0 = ranks[0]
    with pytest.raises(SlowMoError) as e:
        s0.outer_step_external()                      # no local steps taken in this iteration
    assert e.value.status == binding.ESTATE
    common = dict(m_local=2, P=w["P"], pitch=s0.pitch, base="nesterov", buffer_policy="reset", alpha=1.0, beta=0.5,
                  gamma=0.1)
    ptrs = [s.t["x"] for s in ranks]
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_sharded(2, ptrs, ptrs, None, ptrs, ptrs, **common)      # rank >= world
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_sharded(0, ptrs * 9, ptrs * 9, None, ptrs * 9, ptrs * 9, **common)   # 18 GPUs
    assert e.value.status == binding.EINVAL
    with pytest.raises(SlowMoError) as e:
        binding.outer_step_sharded(0, ptrs, ptrs, None, ptrs, ptrs, **dict(common, base="adam"))  # Adam needs v
    assert e.value.status == binding.EINVAL
    for s in ranks:
        s.close()


def test_process_group_wrapper_on_the_gpus_at_hand():
    # one process per GPU over NCCL with peer-mapped state; with a single GPU this runs at world size 1,
    # which still exercises the symmetric-memory allocation, the peer-pointer lists and the fences
    import os
    import socket
    import subprocess
    import sys
    import torch
    n = torch.cuda.device_count()
    world = 1 if n < 2 else (2 if n < 4 else 4)
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = r"""
import os, sys
sys.path.insert(0, %r)
import numpy as np, torch, torch.distributed as dist
rank, world = int(sys.argv[1]), int(sys.argv[2])
torch.cuda.set_device(rank)
assert torch.cuda.current_device() == rank        # every rank on a GPU of its own
os.environ["NCCL_NVLS_ENABLE"] = "0"
dist.init_process_group("nccl", rank=rank, world_size=world, init_method="tcp://127.0.0.1:" + sys.argv[3],
                        device_id=torch.device("cuda", rank))
import oracle
from paper_1910_00643_b200 import workloads
from paper_1910_00643_b200.sharded import ShardedSlowMo
w = workloads.workload("tiny", P=5003, m=4, tau=3, T=3, buffer_policy="average", seed=33)
s = ShardedSlowMo(w)
assert torch.cuda.current_device() == rank and s.local.t["x"].device.index == rank
gammas = (w["gamma"] * np.array([1.0, 0.5, 2.0])).astype(np.float32)      # a learning-rate schedule
for t in range(w["T"]):
    s.set_gamma(float(gammas[t]))
    s.local_steps(w["tau"])
    s.outer_step()
ref = oracle.run(oracle.make_config(**w), j0=0, n=w["P"], precision="f32", gamma_t=gammas)
ml = s.m_local
assert np.array_equal(s.get_params("x").view(np.uint32), ref["x"][rank * ml:(rank + 1) * ml].view(np.uint32))
assert np.array_equal(s.get_params("h").view(np.uint32), ref["h"][rank * ml:(rank + 1) * ml].view(np.uint32))
assert np.array_equal(s.get_params("anchor")[0].view(np.uint32), ref["anchor"].view(np.uint32))
assert np.array_equal(s.get_params("u")[0].view(np.uint32), ref["u"].view(np.uint32))
s.close()
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
""" % root
    procs = [subprocess.Popen([sys.executable, "-c", script, str(r), str(world), str(port)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT) for r in range(world)]
    outs = [p.communicate(timeout=600)[0].decode() for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o[-3000:]
        assert "ok" in o
