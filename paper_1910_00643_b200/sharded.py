"""Workers sharded over the GPUs of one node: one process per GPU, each holding the replica rows
of its own m / world workers, with the outer step's exact average done by
slowmo_outer_step_sharded over peer-mapped memory.

PyTorch provides the plumbing only: torch.distributed (NCCL) for the process group and
torch's symmetric memory for device allocations whose addresses are mapped into every
peer. All arithmetic runs in the library's kernels; peer memory is touched with plain loads and
stores only.
"""
from . import binding
from .binding import SlowMo, round_up


class ShardedSlowMo:
    """m workers over `world` GPUs. Call from every rank of an initialised NCCL process group,
    with the rank's CUDA device current."""

    PEER_TENSORS = ("x", "h", "v", "anchor", "u")

    def __init__(self, workload, group=None):
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm_mem
        self.torch, self.dist = torch, dist
        group = group if group is not None else dist.group.WORLD
        self.group = group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        w = dict(workload)
        if w["m"] % self.world:
            raise ValueError("the number of workers must be a multiple of the number of GPUs")
        if w["base"].startswith("sgp"):
            raise ValueError("push-sum mixing across GPUs is not implemented: use a communication-free base")
        self.m_local = w["m"] // self.world
        self.workload = w
        pitch = round_up(w["P"], 64)
        adam = "adam" in w["base"]
        # state that peers read and write lives in symmetric memory
        self.handles, given = {}, {}
        for name in self.PEER_TENSORS:
            if name == "v" and not adam:
                continue
            rows = 1 if name in ("anchor", "u") else self.m_local
            t = symm_mem.empty(rows * pitch, dtype=torch.float32, device=torch.device("cuda", torch.cuda.current_device()))
            self.handles[name] = symm_mem.rendezvous(t, group)
            given[name] = t
        self.local = SlowMo(dict(w, m=self.m_local, worker_offset=self.rank * self.m_local), pitch=pitch,
                            tensors=given)
        self.pitch = pitch
        self.peers = {name: [int(p) for p in h.buffer_ptrs] for name, h in self.handles.items()}
        self._token = torch.zeros(1, device="cuda")
        self.gamma = w["gamma"]

    def set_gamma(self, gamma):
        """gamma_t of a learning-rate schedule (between outer iterations): used by this GPU's local
        steps and by Eq. (2), (3) in the sharded outer step. Every rank must make the same call."""
        self.local.set_gamma(gamma)
        self.gamma = gamma

    def _fence(self):
        """Stream-ordered meeting point of all GPUs: nothing enqueued after it on the context's
        stream starts before every GPU has finished what it enqueued before it."""
        torch = self.torch
        with torch.cuda.stream(self.local.stream):
            self.dist.all_reduce(self._token, group=self.group)

    def local_steps(self, n):
        self.local.local_steps(n)

    def outer_step(self):
        w = self.workload
        self.local.materialize()        # a deferred or virtual state must be in the rows peers will read
        self._fence()
        binding.outer_step_sharded(
            self.rank, self.peers["x"], self.peers["h"], self.peers.get("v"), self.peers["anchor"], self.peers["u"],
            m_local=self.m_local, P=w["P"], pitch=self.pitch, base=w["base"], buffer_policy=w["buffer_policy"],
            alpha=w["alpha"], beta=w["beta"], gamma=self.gamma, stream=self.local.stream)
        self._fence()
        self.local.outer_step_external()

    def run(self, T):
        for _ in range(T):
            self.local_steps(self.workload["tau"])
            self.outer_step()

    def get_params(self, which, **kw):
        return self.local.get_params(which, **kw)

    def close(self):
        self.local.close()
