"""ctypes binding of libslowmo.so: the same entry points as include/slowmo.h, argument
marshalling only. PyTorch is used for device memory and streams; every step of the method
runs in the library's CUDA kernels.

There is no fallback: if the shared library is missing or a call fails, an exception is
raised.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslowmo.so")

OK, EINVAL, ESTATE, EALIGN, ECUDA, ENOMEM, ETIMEOUT, ENOTIMPL = 0, -1, -2, -3, -4, -5, -6, -7
BASE = {"nesterov": 0, "adam": 1, "sgp_nesterov": 2, "sgp_adam": 3}
POLICY = {"reset": 0, "maintain": 1, "average": 2}
GRAD = {"generated": 0, "supplied": 1}
TENSOR = {"x": 0, "anchor": 1, "u": 2, "h": 3, "v": 4, "a": 5, "c": 6}
KERNEL = {"local": 0, "outer": 1}
VARIANT = {"default": 0, "direct": 1, "staged": 2, "fused": 3, "lazy": 4, "row_tiles": 5, "column_owner": 6}
EXPORTS = ["slowmo_create", "slowmo_destroy", "slowmo_local_steps", "slowmo_outer_step",
           "slowmo_set_gamma", "slowmo_get_params", "slowmo_set_params", "slowmo_get_counters",
           "slowmo_fill_gradient", "slowmo_debug_noise", "slowmo_tensor_range",
           "slowmo_set_variant", "slowmo_sync_status", "slowmo_strerror", "slowmo_last_cuda_error",
           "slowmo_outer_step_static", "slowmo_debug_wait_timeout", "slowmo_iteration_host", "slowmo_materialize",
           "slowmo_outer_step_sharded", "slowmo_outer_step_external",
           "slowmo_debug_words_to_normals", "slowmo_get_state", "slowmo_set_state",
           "slowmo_iteration_host_supplied"]


class SlowMoError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: {strerror(status)} ({status})")


class Config(C.Structure):
    _fields_ = [
        ("P", C.c_uint64), ("m", C.c_uint32), ("tau", C.c_uint32),
        ("alpha", C.c_float), ("beta", C.c_float), ("gamma", C.c_float),
        ("base", C.c_int32), ("mu", C.c_float), ("weight_decay", C.c_float),
        ("adam_b1", C.c_float), ("adam_b2", C.c_float), ("adam_eps", C.c_float),
        ("buffer_policy", C.c_int32), ("grad_mode", C.c_int32),
        ("seed", C.c_uint64),
        ("a_lo", C.c_float), ("a_hi", C.c_float), ("c_std", C.c_float), ("sigma", C.c_float),
        ("x_init", C.c_float),
        ("n_tensors", C.c_uint32), ("tensor_sizes", C.POINTER(C.c_uint64)), ("no_average", C.c_int32),
        ("worker_offset", C.c_uint32),
    ]


class Buffers(C.Structure):
    _fields_ = [("x", C.c_void_p), ("h", C.c_void_p), ("v", C.c_void_p), ("anchor", C.c_void_p),
                ("u", C.c_void_p), ("a", C.c_void_p), ("c", C.c_void_p), ("pitch", C.c_uint64)]


class ShardArgs(C.Structure):
    _fields_ = [("world", C.c_uint32), ("rank", C.c_uint32), ("m_local", C.c_uint32),
                ("P", C.c_uint64), ("pitch", C.c_uint64),
                ("x", C.POINTER(C.c_void_p)), ("h", C.POINTER(C.c_void_p)), ("v", C.POINTER(C.c_void_p)),
                ("anchor", C.POINTER(C.c_void_p)), ("u", C.POINTER(C.c_void_p)),
                ("base", C.c_int32), ("buffer_policy", C.c_int32),
                ("alpha", C.c_float), ("beta", C.c_float), ("gamma_t", C.c_float)]


class State(C.Structure):
    _fields_ = [("t", C.c_uint64), ("l", C.c_uint64), ("k", C.c_uint32), ("gamma_t", C.c_float)]


_lib = None


def lib():
    """Load libslowmo.so (once). Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # not built yet: compile it now (nvcc, sm_100a); one process at a time
            import fcntl
            from . import build as _build
            try:
                with open(os.path.join(_HERE, ".build.lock"), "w") as lock:
                    fcntl.flock(lock, fcntl.LOCK_EX)
                    if not os.path.exists(LIB_PATH):
                        _build.build(force=True)
            except Exception as exc:
                raise ImportError(f"{LIB_PATH} is missing and could not be built with nvcc: {exc}") from exc
        L = C.CDLL(LIB_PATH)
        vp, u64, u32, i32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int32
        sig = {
            "slowmo_create": [C.POINTER(Config), C.POINTER(Buffers), vp, C.POINTER(vp)],
            "slowmo_destroy": [vp],
            "slowmo_local_steps": [vp, u32, vp],
            "slowmo_outer_step": [vp],
            "slowmo_set_gamma": [vp, C.c_float],
            "slowmo_get_params": [vp, C.c_int, i32, u64, u64, vp, C.c_int],
            "slowmo_set_params": [vp, C.c_int, i32, u64, u64, vp, C.c_int],
            "slowmo_get_counters": [vp, C.POINTER(u64), C.POINTER(u32), C.POINTER(u64)],
            "slowmo_fill_gradient": [vp, vp],
            "slowmo_debug_noise": [vp, u32, u64, u32, u32, u64, u64, vp, vp],
            "slowmo_tensor_range": [vp, u32, C.POINTER(u64), C.POINTER(u64)],
            "slowmo_set_variant": [vp, C.c_int, C.c_int],
            "slowmo_sync_status": [vp],
            "slowmo_last_cuda_error": [vp],
            "slowmo_debug_wait_timeout": [vp, u32],
            "slowmo_iteration_host": [vp, vp, vp, u32],
            "slowmo_iteration_host_supplied": [vp, vp, vp, vp, u32],
            "slowmo_materialize": [vp],
            "slowmo_outer_step_sharded": [C.POINTER(ShardArgs), vp],
            "slowmo_outer_step_external": [vp],
            "slowmo_debug_words_to_normals": [vp, vp, u64, vp],
            "slowmo_get_state": [vp, C.POINTER(State)],
            "slowmo_set_state": [vp, C.POINTER(State)],
            "slowmo_outer_step_static": [vp, vp, vp, vp, vp, u64, u64, u32, i32, i32, C.c_float, C.c_float,
                                         C.c_float, vp, C.c_int],
        }
        for name, args in sig.items():
            f = getattr(L, name)
            f.argtypes = args
            f.restype = C.c_int
        L.slowmo_strerror.argtypes = [C.c_int]
        L.slowmo_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def strerror(status):
    return lib().slowmo_strerror(status).decode()


def _check(status, what):
    if status != OK:
        raise SlowMoError(status, what)


def make_config(*, P, m, tau, alpha=1.0, beta=0.0, gamma=0.1, base="nesterov", mu=0.0, weight_decay=0.0,
                adam_b1=0.9, adam_b2=0.999, adam_eps=1e-8, buffer_policy="reset", grad_mode="generated",
                seed=0, a_lo=0.5, a_hi=2.0, c_std=1.0, sigma=0.0, x_init=0.0, tensor_sizes=None, no_average=False,
                worker_offset=0, **_ignored):
    """Fill the C config from paper-notation keyword arguments (see include/slowmo.h)."""
    cfg = Config(P, m, tau, alpha, beta, gamma, BASE[base] if isinstance(base, str) else base, mu,
                 weight_decay, adam_b1, adam_b2, adam_eps,
                 POLICY[buffer_policy] if isinstance(buffer_policy, str) else buffer_policy,
                 GRAD[grad_mode] if isinstance(grad_mode, str) else grad_mode, seed, a_lo, a_hi, c_std,
                 sigma, x_init, 0, None, 1 if no_average else 0, worker_offset)
    if tensor_sizes is not None:
        arr = (C.c_uint64 * len(tensor_sizes))(*[int(s) for s in tensor_sizes])
        cfg._keep = arr
        cfg.n_tensors = len(tensor_sizes)
        cfg.tensor_sizes = C.cast(arr, C.POINTER(C.c_uint64))
    return cfg


def outer_step_static(x, h, v, anchor, u, *, pitch, P, m, base, buffer_policy, alpha, beta, gamma,
                      stream=None, wait=True):
    """slowmo_outer_step_static: the outer step on caller-owned torch CUDA tensors, for callers
    that may not allocate device memory (no context, no cudaMalloc). Raises on any error."""
    ptr = lambda t: None if t is None else t.data_ptr()
    rc = lib().slowmo_outer_step_static(ptr(x), ptr(h), ptr(v), ptr(anchor), ptr(u), pitch, P, m,
                                        BASE[base] if isinstance(base, str) else base,
                                        POLICY[buffer_policy] if isinstance(buffer_policy, str) else buffer_policy,
                                        alpha, beta, gamma, None if stream is None else stream.cuda_stream,
                                        1 if wait else 0)
    _check(rc, "slowmo_outer_step_static")


def outer_step_sharded(rank, x, h, v, anchor, u, *, m_local, P, pitch, base, buffer_policy, alpha, beta, gamma,
                       stream=None):
    """slowmo_outer_step_sharded for GPU `rank`: x, h, v, anchor, u are lists (one entry per GPU) of
    device pointers (ints) or torch tensors, valid on the calling GPU."""
    world = len(x)
    ptr = lambda t: t if isinstance(t, int) or t is None else t.data_ptr()
    arr = lambda lst: None if lst is None else (C.c_void_p * world)(*[ptr(t) for t in lst])
    keep = [arr(x), arr(h), arr(v), arr(anchor), arr(u)]
    cast = lambda a: None if a is None else C.cast(a, C.POINTER(C.c_void_p))
    args = ShardArgs(world, rank, m_local, P, pitch, cast(keep[0]), cast(keep[1]), cast(keep[2]), cast(keep[3]),
                     cast(keep[4]), BASE[base] if isinstance(base, str) else base,
                     POLICY[buffer_policy] if isinstance(buffer_policy, str) else buffer_policy, alpha, beta, gamma)
    _check(lib().slowmo_outer_step_sharded(C.byref(args), None if stream is None else stream.cuda_stream),
           "slowmo_outer_step_sharded")


def round_up(n, q):
    return (n + q - 1) // q * q


class SlowMo:
    """One SlowMo context with its device tensors (torch-allocated) on the current device.

    Methods carry the names of the C entry points without the prefix and do nothing but
    marshal arguments.
    """

    def __init__(self, workload, stream=None, pitch=None, guard=0, tensors=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("libslowmo needs a CUDA device (sm_100a); there is no CPU path")
        self.torch = torch
        w = dict(workload)
        if w.get("n_tensors") and "tensor_sizes" not in w:
            from .workloads import tensor_sizes
            w["tensor_sizes"] = tensor_sizes(w["P"], w["n_tensors"], w.get("seed", 0))
        self.workload = w
        self.cfg = make_config(**w)
        self.P, self.m, self.tau = w["P"], w["m"], w["tau"]
        self.pitch = pitch if pitch is not None else round_up(self.P, 64)  # 256-byte rows: measured faster than 128
        self.stream = stream if stream is not None else torch.cuda.Stream()
        self.guard = guard
        adam = self.cfg.base in (BASE["adam"], BASE["sgp_adam"])
        generated = self.cfg.grad_mode == GRAD["generated"]
        self._raw = {}
        self.t = {}
        self._given = tensors or {}   # caller-allocated tensors (e.g. peer-mapped memory), by name
        self.outer_rows = self.m if self.cfg.no_average else 1
        for name, rows, need in (("x", self.m, True), ("h", self.m, True), ("v", self.m, adam),
                                 ("anchor", self.outer_rows, True), ("u", self.outer_rows, True),
                                 ("a", 1, generated),
                                 ("c", self.m, generated)):
            self.t[name] = self._alloc(name, rows) if need else None
        ptr = lambda k: self.t[k].data_ptr() if self.t[k] is not None else None
        self.buf = Buffers(ptr("x"), ptr("h"), ptr("v"), ptr("anchor"), ptr("u"), ptr("a"), ptr("c"), self.pitch)
        self.grad = None
        self.ctx = C.c_void_p()
        # creation enqueues fills on self.stream; order it after the allocations' stream
        self.stream.wait_stream(torch.cuda.current_stream())
        _check(lib().slowmo_create(C.byref(self.cfg), C.byref(self.buf), self.stream.cuda_stream,
                                   C.byref(self.ctx)), "slowmo_create")

    # guard words before and after every tensor let tests detect out-of-bounds writes
    GUARD_VALUE = -12345.5

    def _alloc(self, name, rows):
        torch = self.torch
        n = rows * self.pitch
        if name in self._given:
            t = self._given[name]
            assert t.is_cuda and t.dtype == torch.float32 and t.numel() >= n and t.data_ptr() % 16 == 0, name
            return t.view(-1)[:n]
        g = self.guard
        raw = torch.empty(n + 2 * g, dtype=torch.float32, device="cuda")
        if g:
            raw[:g] = self.GUARD_VALUE
            raw[g + n:] = self.GUARD_VALUE
        self._raw[name] = raw
        return raw[g:g + n]

    def guards_intact(self):
        g = self.guard
        self.synchronize()
        for name, raw in self._raw.items():
            n = raw.numel() - 2 * g
            if g and not (bool((raw[:g] == self.GUARD_VALUE).all()) and bool((raw[g + n:] == self.GUARD_VALUE).all())):
                return False
        return True

    def alloc_gradient(self):
        """Device [m, pitch] tensor for supplied-gradient mode (kept as self.grad)."""
        self.grad = self._alloc("grad", self.m)
        return self.grad

    def fill_gradient(self, grad=None):
        grad = self.grad if grad is None else grad
        _check(lib().slowmo_fill_gradient(self.ctx, grad.data_ptr()), "slowmo_fill_gradient")

    def local_steps(self, n, grad=None):
        _check(lib().slowmo_local_steps(self.ctx, n, None if grad is None else grad.data_ptr()),
               "slowmo_local_steps")

    def outer_step(self):
        _check(lib().slowmo_outer_step(self.ctx), "slowmo_outer_step")

    def iteration_host(self, c_host, anchor_host, chunks=8):
        """slowmo_iteration_host: one outer iteration with host input c [m, P] and host output
        anchor (torch CPU tensors, pinned for overlap, or numpy arrays)."""
        ptr = lambda a: a.ctypes.data if isinstance(a, np.ndarray) else a.data_ptr()
        _check(lib().slowmo_iteration_host(self.ctx, ptr(c_host), ptr(anchor_host), chunks), "slowmo_iteration_host")

    def iteration_host_supplied(self, grad_host, anchor_host, chunks=8, grad_dev=None):
        """slowmo_iteration_host_supplied: one outer iteration with the host gradient grad_host [m, P]
        staged through the device tensor grad_dev (default: the context's gradient buffer)."""
        grad_dev = self.grad if grad_dev is None else grad_dev
        ptr = lambda a: a.ctypes.data if isinstance(a, np.ndarray) else a.data_ptr()
        _check(lib().slowmo_iteration_host_supplied(self.ctx, ptr(grad_host), grad_dev.data_ptr(), ptr(anchor_host),
                                                    chunks), "slowmo_iteration_host_supplied")

    def outer_step_external(self):
        _check(lib().slowmo_outer_step_external(self.ctx), "slowmo_outer_step_external")

    def materialize(self):
        _check(lib().slowmo_materialize(self.ctx), "slowmo_materialize")

    def set_gamma(self, gamma):
        _check(lib().slowmo_set_gamma(self.ctx, gamma), "slowmo_set_gamma")

    def set_variant(self, kernel, variant):
        _check(lib().slowmo_set_variant(self.ctx, KERNEL[kernel], VARIANT[variant]), "slowmo_set_variant")

    def sync_status(self):
        _check(lib().slowmo_sync_status(self.ctx), "slowmo_sync_status")

    def debug_wait_timeout(self, tries=4096):
        _check(lib().slowmo_debug_wait_timeout(self.ctx, tries), "slowmo_debug_wait_timeout")

    def counters(self):
        t, k, l = C.c_uint64(), C.c_uint32(), C.c_uint64()
        _check(lib().slowmo_get_counters(self.ctx, C.byref(t), C.byref(k), C.byref(l)), "slowmo_get_counters")
        return t.value, k.value, l.value

    def get_state(self):
        """slowmo_get_state: position in Algorithm 1 as a dict(t, k, l, gamma_t)."""
        st = State()
        _check(lib().slowmo_get_state(self.ctx, C.byref(st)), "slowmo_get_state")
        return {"t": st.t, "k": st.k, "l": st.l, "gamma_t": st.gamma_t}

    def set_state(self, t, k, l, gamma_t):
        st = State(t, l, k, gamma_t)
        _check(lib().slowmo_set_state(self.ctx, C.byref(st)), "slowmo_set_state")

    def get_params(self, which, replica=-1, offset=0, count=None, out=None):
        """Copy columns [offset, offset+count) of tensor `which` to host (numpy) or to `out`
        (a torch CUDA tensor or pinned/pageable numpy array)."""
        count = self.P - offset if count is None else count
        one_row = which == "a" or (which in ("anchor", "u") and not self.cfg.no_average)
        rows = 1 if (replica >= 0 or one_row) else self.m
        on_device = 0
        if out is None:
            out = np.empty((rows, count), np.float32)
            dst = out.ctypes.data
        elif isinstance(out, np.ndarray):
            dst = out.ctypes.data
        else:
            dst = out.data_ptr()
            on_device = 1 if out.is_cuda else 0
        _check(lib().slowmo_get_params(self.ctx, TENSOR[which], replica, offset, count, dst, on_device),
               "slowmo_get_params")
        return out

    def set_params(self, which, src, replica=-1, offset=0, count=None):
        count = self.P - offset if count is None else count
        if isinstance(src, np.ndarray):
            assert src.dtype == np.float32 and src.flags.c_contiguous
            ptr, on_device = src.ctypes.data, 0
        else:
            ptr, on_device = src.data_ptr(), 1 if src.is_cuda else 0
        _check(lib().slowmo_set_params(self.ctx, TENSOR[which], replica, offset, count, ptr, on_device),
               "slowmo_set_params")

    def debug_noise(self, tag, t, k, w, j0, n, words=True, normals=True):
        torch = self.torch
        with torch.cuda.stream(self.stream):
            wd = torch.empty(n, dtype=torch.int64, device="cuda") if words else None
            z = torch.empty(n, dtype=torch.float32, device="cuda") if normals else None
        _check(lib().slowmo_debug_noise(self.ctx, tag, t, k, w, j0, n, wd.data_ptr() if words else None,
                                        z.data_ptr() if normals else None), "slowmo_debug_noise")
        self.synchronize()
        return (wd.cpu().numpy().view(np.uint64) if words else None, z.cpu().numpy() if normals else None)

    def debug_words_to_normals(self, words):
        """Both normals of each 64-bit word (numpy uint64 array) -> float32 [n, 2]."""
        torch = self.torch
        w = torch.from_numpy(np.ascontiguousarray(words, dtype=np.uint64).view(np.int64)).cuda()
        out = torch.empty(2 * w.numel(), dtype=torch.float32, device="cuda")
        self.stream.wait_stream(torch.cuda.current_stream())
        _check(lib().slowmo_debug_words_to_normals(self.ctx, w.data_ptr(), w.numel(), out.data_ptr()),
               "slowmo_debug_words_to_normals")
        self.synchronize()
        return out.cpu().numpy().reshape(-1, 2)

    def tensor_range(self, idx):
        off, cnt = C.c_uint64(), C.c_uint64()
        _check(lib().slowmo_tensor_range(self.ctx, idx, C.byref(off), C.byref(cnt)), "slowmo_tensor_range")
        return off.value, cnt.value

    def run(self, T, grad=None):
        """T outer iterations of Algorithm 1: tau local steps, then the outer step."""
        for _ in range(T):
            self.local_steps(self.tau, grad)
            self.outer_step()

    def synchronize(self):
        self.stream.synchronize()

    def close(self):
        if self.ctx:
            _check(lib().slowmo_destroy(self.ctx), "slowmo_destroy")
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
