"""Host-side checks that need no GPU: the shared library builds, loads and exports every
symbol the header declares; argument validation answers before any CUDA call; the workload
descriptions are consistent; the benchmark's multi-rank aggregation works over gloo."""
import ctypes as C
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_1910_00643_b200 import build, binding
    build.build()
    return binding


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "slowmo.h")).read()
    declared = set(re.findall(r"\b(slowmo_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert binding.strerror(0) == "ok" and "aligned" in binding.strerror(binding.EALIGN)


def test_struct_layouts_match_the_header(binding, tmp_path):
    # sizes and offsets as the C compiler lays out include/slowmo.h
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "slowmo.h"\n'
        'int main(void){printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof(slowmo_config), '
        'offsetof(slowmo_config, seed), offsetof(slowmo_config, x_init), offsetof(slowmo_config, tensor_sizes), '
        'sizeof(slowmo_buffers), offsetof(slowmo_buffers, a), offsetof(slowmo_buffers, pitch));return 0;}\n')
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    want = [int(v) for v in subprocess.check_output([str(exe)]).split()]
    got = [C.sizeof(binding.Config), binding.Config.seed.offset, binding.Config.x_init.offset,
           binding.Config.tensor_sizes.offset, C.sizeof(binding.Buffers), binding.Buffers.a.offset,
           binding.Buffers.pitch.offset]
    assert got == want


def _create(binding, buf_overrides=None, **cfg_overrides):
    from paper_1910_00643_b200 import workloads
    w = workloads.workload("tiny")
    w.update(cfg_overrides)
    cfg = binding.make_config(**w)
    fake = 0x7F0000000000  # never dereferenced: validation fails first
    b = dict(x=fake, h=fake, v=fake, anchor=fake, u=fake, a=fake, c=fake, pitch=4096)
    b.update(buf_overrides or {})
    buf = binding.Buffers(b["x"], b["h"], b["v"], b["anchor"], b["u"], b["a"], b["c"], b["pitch"])
    ctx = C.c_void_p()
    rc = binding.lib().slowmo_create(C.byref(cfg), C.byref(buf), None, C.byref(ctx))
    assert not ctx.value or rc == 0
    return rc


@pytest.mark.parametrize("bad", [
    dict(P=0), dict(m=0), dict(tau=0), dict(gamma=0.0), dict(gamma=-1.0), dict(gamma=float("inf")),
    dict(gamma=float("nan")), dict(beta=1.0), dict(beta=-0.1), dict(alpha=0.0), dict(base=7),
    dict(buffer_policy=3), dict(grad_mode=2), dict(mu=1.0), dict(weight_decay=-1.0),
    dict(base="adam", adam_b1=1.0), dict(base="adam", adam_b2=-0.5), dict(base="adam", adam_eps=0.0),
    dict(sigma=-1.0), dict(a_lo=2.0, a_hi=1.0), dict(P=2**35), dict(P=2**34 - 16383), dict(tensor_sizes=[4000, 97]),
    dict(tensor_sizes=[4096, 0]),
])
def test_create_rejects_bad_configurations(binding, bad):
    assert _create(binding, **bad) == binding.EINVAL


def test_parameter_count_limit(binding):
    # one parameter more than SLOWMO_MAX_P is refused even when the rows are long enough
    assert _create(binding, dict(pitch=2**34), P=2**34 - 16383) == binding.EINVAL
    # so is a worker count whose row tiles no longer fit one grid dimension
    assert _create(binding, dict(pitch=2**33), P=2**33, m=2**9) == binding.EINVAL


def test_create_rejects_bad_buffers(binding):
    assert _create(binding, dict(x=None)) == binding.EINVAL
    assert _create(binding, dict(a=None)) == binding.EINVAL          # generated mode needs a and c
    assert _create(binding, dict(v=None), base="adam") == binding.EINVAL
    assert _create(binding, dict(pitch=4094)) == binding.EALIGN
    assert _create(binding, dict(pitch=4092)) == binding.EINVAL      # pitch < P
    assert _create(binding, dict(u=0x7F0000000004)) == binding.EALIGN
    assert binding.lib().slowmo_create(None, None, None, None) == binding.EINVAL


def test_null_context_is_an_error_everywhere(binding):
    L = binding.lib()
    assert L.slowmo_local_steps(None, 1, None) == binding.EINVAL
    assert L.slowmo_outer_step(None) == binding.EINVAL
    assert L.slowmo_set_gamma(None, 0.1) == binding.EINVAL
    assert L.slowmo_get_params(None, 0, -1, 0, 1, None, 0) == binding.EINVAL
    assert L.slowmo_destroy(None) == binding.EINVAL
    assert L.slowmo_sync_status(None) == binding.EINVAL


def test_no_cpu_fallback(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_1910_00643_b200 import SlowMo, workloads
    with pytest.raises(RuntimeError):
        SlowMo(workloads.workload("tiny"))
    # a valid configuration reaches the CUDA runtime and reports its failure
    assert _create(binding) == binding.ECUDA


def test_product_code_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_1910_00643_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text, f
                assert "slowmo_oracle" not in text, f


def test_workload_descriptions():
    from paper_1910_00643_b200 import workloads
    from bench import (fused_outer_step_bytes, lazy_outer_step_bytes, local_step_bytes, outer_step_bytes,
                       virtual_first_step_bytes)
    w = workloads.workload("resnet50")
    sizes = workloads.tensor_sizes(w["P"], w["n_tensors"], w["seed"])
    assert len(sizes) == 161 and int(sizes.sum()) == w["P"] and sizes.min() >= 1
    assert sizes.max() / max(1, np.median(sizes)) > 20          # heavy tail
    assert np.array_equal(sizes, workloads.tensor_sizes(w["P"], 161, 0))  # seeded
    # algorithmic bytes per unit (replica-parameter update / parameter)
    assert local_step_bytes(w) / (w["m"] * w["P"]) == pytest.approx(20.125)
    assert outer_step_bytes(w) / w["P"] == 528
    assert outer_step_bytes(workloads.workload("bmuf")) / w["P"] == 208
    assert outer_step_bytes(workloads.workload("sync_sgd")) / w["P"] == 272
    wa = workloads.workload("transformer_adam")
    assert local_step_bytes(wa) / (wa["m"] * wa["P"]) == pytest.approx(28.5)
    assert outer_step_bytes(wa) / wa["P"] == 80
    ws = workloads.workload("stress_tau12")
    assert local_step_bytes(ws) / (ws["m"] * ws["P"]) == 20
    assert outer_step_bytes(ws) / ws["P"] == 64
    # outer step with the last inner step fused in: 20m + 16 (+4 for a) per parameter, +8m for Adam's v
    assert fused_outer_step_bytes(ws) / ws["P"] == 96
    assert fused_outer_step_bytes(w) / w["P"] == 20 * 32 + 20
    assert fused_outer_step_bytes(wa) / wa["P"] == 28 * 8 + 20
    # lazy variant: no broadcast rows, no reset / averaged buffer rows; the next step reads the anchor
    assert lazy_outer_step_bytes(w) / w["P"] == 12 * 32 + 20 + 4            # average: + one row of means
    assert virtual_first_step_bytes(w) / w["P"] == 12 * 32 + 8 + 4
    assert lazy_outer_step_bytes(ws) / ws["P"] == 12 * 4 + 16               # reset, supplied
    assert virtual_first_step_bytes(ws) / ws["P"] == 12 * 4 + 4
    assert lazy_outer_step_bytes(wa) / wa["P"] == 16 * 8 + 20 + 8 * 8       # maintain keeps the buffer rows
    j = workloads.sample_coordinates(10**9, 1000, seed=1)
    assert j[0] == 0 and j[-1] == 10**9 - 1 and len(np.unique(j)) == len(j)


_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", rank=int(sys.argv[1]), world_size=2,
                        init_method="tcp://127.0.0.1:" + sys.argv[2])
rank = dist.get_rank()
value, ms = bench.aggregate_throughput(1000.0 * (rank + 1), 10.0 * (rank + 1))
bench.barrier()
assert ms == 20.0, ms
assert abs(value - 3000.0 / 0.020) < 1e-6, value
print("rank", rank, "ok")
dist.destroy_process_group()
"""


def test_two_rank_aggregation_over_gloo(tmp_path):
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = str(sk.getsockname()[1])
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    procs = [subprocess.Popen([sys.executable, str(script), str(r), port], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT) for r in range(2)]
    outs = [p.communicate(timeout=180)[0].decode() for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "ok" in o


def test_gpus_flag_starts_the_ranks_itself(tmp_path):
    # `bench.py --gpus 2` without a launcher re-executes itself under torch.distributed.run with two
    # ranks on 127.0.0.1; the host-only self-test stands in for the GPU arm (gloo, no device)
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-ranks"],
                         capture_output=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr.decode()[-2000:]
    lines = [l for l in out.stdout.decode().splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout.decode()
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["ms"] == 20.0 and abs(line["value"] - 3000.0 / 0.020) < 1e-6
    # one rank needs no launcher
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--selftest-ranks"], capture_output=True,
                         timeout=120, env=env)
    assert out.returncode == 0 and json.loads(out.stdout.decode().strip())["n_gpus"] == 1
    # under a launcher that started another number of ranks the mismatch is an error, not a silent 1-GPU run
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-ranks"],
                         capture_output=True, timeout=120, env=dict(env, WORLD_SIZE="3", RANK="0"))
    assert out.returncode != 0 and b"WORLD_SIZE=3" in out.stderr
    import bench
    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "2"])
    assert "--nproc-per-node=4" in cmd and "127.0.0.1" in cmd and cmd[-4:] == ["--gpus", "4", "--steps", "2"]


def test_traffic_ratios_come_from_the_committed_profiles():
    # every ratio bench.py reports is read from a `traffic_ratio:` line of an ncu summary under profiles/
    # taken on the current kernel sources; nothing is hard-coded
    import bench
    ratios = bench.traffic_ratios()
    text = "".join(open(os.path.join(ROOT, "profiles", f)).read() for f in os.listdir(os.path.join(ROOT, "profiles")))
    for case, (ratio, source) in ratios.items():
        assert f"case={case} " in text and 0.5 < ratio < 1.5 and source.endswith(".md")
    assert len(bench.kernel_source_hash()) == 12


def test_reference_arm_runs_on_the_host():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--reference-coords", "2048"], capture_output=True, timeout=300)
    assert out.returncode == 0, out.stderr.decode()
    import json
    line = json.loads(out.stdout.decode().strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
