"""ctypes binding of ``libevo.so`` (declared in ``include/evo.h``).

Argument marshalling only: every step of ask / rollout / tell runs in the library's CUDA
kernels.  PyTorch supplies device memory (the workspace, fitness and trace buffers) and the
stream.  There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import workloads as W

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libevo.so")
LIB_DEBUG_PATH = os.path.join(_HERE, "libevo_debug.so")     # checked build (-DEVO_DEBUG)

EVO_MAX_LAYERS = 8
STATUS = {0: "EVO_OK", 1: "EVO_ERR_INVALID_ARG", 2: "EVO_ERR_BAD_ORDER", 3: "EVO_ERR_WORKSPACE",
          4: "EVO_ERR_CUDA", 5: "EVO_ERR_NONFINITE", 6: "EVO_ERR_TIMEOUT", 7: "EVO_ERR_UNSUPPORTED"}
ROLLOUT_AUTO, ROLLOUT_GENERIC, ROLLOUT_TILED = 0, 1, 2
DEBUG_DROP_COMPLETION = 1


class EvoConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("pop_size", C.c_uint32), ("seed", C.c_uint64),
        ("param_dim", C.c_uint32), ("noise_mode", C.c_uint32),
        ("sigma", C.c_float), ("lr", C.c_float),
        ("beta1", C.c_float), ("beta2", C.c_float), ("adam_eps", C.c_float),
        ("policy_kind", C.c_uint32), ("n_layers", C.c_uint32),
        ("layer_sizes", C.c_uint32 * (EVO_MAX_LAYERS + 1)), ("action_scale", C.c_float),
        ("task_kind", C.c_uint32), ("episodes", C.c_uint32), ("horizon", C.c_uint32),
        ("batch", C.c_uint32), ("trace_steps", C.c_uint32), ("rollout_kernel", C.c_uint32),
        ("task_param", C.c_float * 16),
        ("optimizer", C.c_uint32), ("clipup_momentum", C.c_float), ("clipup_max_speed", C.c_float),
        ("sigma_mode", C.c_uint32), ("sigma_lr", C.c_float), ("sigma_max_change", C.c_float),
        ("shard_first_pair", C.c_uint32), ("shard_pairs", C.c_uint32),
        ("wait_cycles_log2", C.c_uint32), ("debug_flags", C.c_uint32),
    ]


class EvoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)}")


_lib = None
_lib_debug = None


def load_library(debug: bool = False):
    """Loads libevo.so (or the checked build libevo_debug.so); raises if it has not been built
    (no CPU fallback exists)."""
    global _lib, _lib_debug
    if debug and _lib_debug is not None:
        return _lib_debug
    if not debug and _lib is not None:
        return _lib
    path = LIB_DEBUG_PATH if debug else LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} is missing: build it with `python -m paper_2202_05008_b200.build`")
    L = C.CDLL(path)
    vp, u32p, szp = C.c_void_p, C.POINTER(C.c_uint32), C.POINTER(C.c_size_t)
    cfgp = C.POINTER(EvoConfig)
    L.evo_workspace_bytes.argtypes = [cfgp, szp]
    L.evo_create.argtypes = [cfgp, vp, C.c_size_t, vp, C.POINTER(vp)]
    L.evo_ask.argtypes = [vp, C.POINTER(vp), szp]
    L.evo_rollout.argtypes = [vp, vp, vp, vp]
    L.evo_tell.argtypes = [vp, vp]
    L.evo_tell_begin.argtypes = [vp, vp]
    L.evo_get_reduce_buffers.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), szp]
    L.evo_tell_end.argtypes = [vp]
    L.evo_set_target.argtypes = [vp, vp]
    L.evo_destroy.argtypes = [vp]
    L.evo_set_batch.argtypes = [vp, vp, vp]
    L.evo_get_center.argtypes = [vp, C.POINTER(vp)]
    L.evo_get_moments.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
    L.evo_get_gradient.argtypes = [vp, C.POINTER(vp)]
    L.evo_get_ranks.argtypes = [vp, C.POINTER(vp), C.POINTER(vp)]
    L.evo_get_eps.argtypes = [vp, C.POINTER(vp)]
    L.evo_get_sigma.argtypes = [vp, C.POINTER(vp)]
    L.evo_set_sigma.argtypes = [vp, vp]
    L.evo_get_counters.argtypes = [vp, u32p, u32p]
    L.evo_set_state.argtypes = [vp, vp, vp, vp, C.c_uint32, C.c_uint32]
    L.evo_sync_status.argtypes = [vp]
    L.evo_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
    L.evo_es_gradient_static.argtypes = [vp, vp, C.c_uint32, C.c_uint32, C.c_size_t, C.c_float, vp, vp]
    L.evo_es_gradient_static.restype = C.c_int
    L.evo_status_string.argtypes = [C.c_int]
    L.evo_status_string.restype = C.c_char_p
    L.evo_version.restype = C.c_uint32
    for name in ("evo_workspace_bytes", "evo_create", "evo_ask", "evo_rollout", "evo_tell", "evo_tell_begin",
                 "evo_get_reduce_buffers", "evo_tell_end", "evo_set_target",
                 "evo_destroy", "evo_set_batch", "evo_get_center", "evo_get_moments",
                 "evo_get_gradient", "evo_get_ranks", "evo_get_eps", "evo_get_sigma", "evo_set_sigma", "evo_get_counters",
                 "evo_set_state", "evo_sync_status", "evo_launch_count"):
        getattr(L, name).restype = C.c_int
    L.evo_debug_check.argtypes = [vp, C.POINTER(C.c_int32), u32p, C.POINTER(C.c_uint64)]
    L.evo_debug_check.restype = C.c_int
    if debug:
        _lib_debug = L
    else:
        _lib = L
    return L


def make_config(w: W.Workload, *, trace_steps: int = 0, rollout_kernel: int = ROLLOUT_AUTO,
                noise_mode: Optional[int] = None, shard_first_pair: int = 0, shard_pairs: int = 0,
                wait_cycles_log2: int = 0, debug_flags: int = 0) -> EvoConfig:
    c = EvoConfig()
    c.struct_size = C.sizeof(EvoConfig)
    c.pop_size, c.param_dim, c.seed = w.pop_size, w.param_dim, w.seed
    c.noise_mode = w.noise_mode if noise_mode is None else noise_mode
    c.sigma, c.lr = w.sigma, w.lr
    c.policy_kind = w.policy_kind
    c.n_layers = max(len(w.layer_sizes) - 1, 0)
    for i, s in enumerate(w.layer_sizes):
        c.layer_sizes[i] = s
    c.action_scale = w.action_scale
    c.task_kind, c.episodes, c.horizon, c.batch = w.task_kind, w.episodes, w.horizon, w.batch
    c.trace_steps, c.rollout_kernel = trace_steps, rollout_kernel
    for i, v in enumerate(w.task_param):
        c.task_param[i] = v
    c.optimizer, c.clipup_momentum, c.clipup_max_speed = w.optimizer, w.clipup_momentum, w.clipup_max_speed
    c.sigma_mode, c.sigma_lr, c.sigma_max_change = w.sigma_mode, w.sigma_lr, w.sigma_max_change
    c.shard_first_pair, c.shard_pairs = shard_first_pair, shard_pairs
    c.wait_cycles_log2, c.debug_flags = wait_cycles_log2, debug_flags
    return c


def _check(code: int, where: str):
    if code != 0:
        raise EvoError(code, where)


class Solver:
    """One ES solver bound to a CUDA device, a stream and a caller-owned workspace tensor."""

    def __init__(self, workload: W.Workload, device="cuda:0", stream: Optional[torch.cuda.Stream] = None,
                 debug: bool = False, **cfg_kw):
        self.lib = load_library(debug)
        self.workload = workload
        self.cfg = make_config(workload, **cfg_kw)
        self.device = torch.device(device)
        nbytes = C.c_size_t(0)
        _check(self.lib.evo_workspace_bytes(C.byref(self.cfg), C.byref(nbytes)), "evo_workspace_bytes")
        self.workspace_bytes = nbytes.value
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
            self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            h = C.c_void_p()
            _check(self.lib.evo_create(C.byref(self.cfg), self._ws_ptr, self.workspace_bytes,
                                       self.stream.cuda_stream, C.byref(h)), "evo_create")
        self._h = h
        # P = members this solver samples and evaluates (its shard); P_global = the population ranked
        self.P_global = workload.pop_size
        self.P, self.D = (2 * self.cfg.shard_pairs if self.cfg.shard_pairs else workload.pop_size), workload.param_dim
        self.ldD = (self.D + 31) // 32 * 32
        self._batch = None

    # -- the five calls ------------------------------------------------------------------
    def ask(self) -> torch.Tensor:
        """theta[P][D] as a strided view (row pitch ldD) of the workspace."""
        p, ld = C.c_void_p(), C.c_size_t()
        _check(self.lib.evo_ask(self._h, C.byref(p), C.byref(ld)), "evo_ask")
        return self._view_f32(p.value, self.P, ld.value)[:, :self.D]

    def rollout(self, theta: Optional[torch.Tensor] = None, fitness: Optional[torch.Tensor] = None,
                trace: Optional[torch.Tensor] = None) -> torch.Tensor:
        if fitness is None:
            fitness = torch.empty(self.P, dtype=torch.float32, device=self.device)
        tp = None
        if theta is not None:
            assert theta.dtype == torch.float32 and theta.is_cuda and theta.stride(1) == 1
            assert theta.shape[0] == self.P and theta.stride(0) == self.ldD
            tp = theta.data_ptr()
        _check(self.lib.evo_rollout(self._h, tp, fitness.data_ptr(),
                                    None if trace is None else trace.data_ptr()), "evo_rollout")
        return fitness

    def tell(self, fitness: torch.Tensor) -> None:
        assert fitness.dtype == torch.float32 and fitness.is_cuda and fitness.numel() == self.P_global
        _check(self.lib.evo_tell(self._h, fitness.data_ptr()), "evo_tell")

    # -- sharded tell: begin -> (caller sums the reduce buffers over the shards) -> end ------------
    def tell_begin(self, fitness_all: torch.Tensor) -> None:
        assert fitness_all.dtype == torch.float32 and fitness_all.is_cuda and fitness_all.numel() == self.P_global
        _check(self.lib.evo_tell_begin(self._h, fitness_all.data_ptr()), "evo_tell_begin")

    def reduce_buffers(self):
        """(grad_sum fp64 [ldD], sigma_sum fp32 [ldD] or None): views to be summed over the shards in place."""
        g, sg, n = C.c_void_p(), C.c_void_p(), C.c_size_t()
        _check(self.lib.evo_get_reduce_buffers(self._h, C.byref(g), C.byref(sg), C.byref(n)), "evo_get_reduce_buffers")
        off = g.value - self.workspace.data_ptr()
        grad = self.workspace[off:off + n.value * 8].view(torch.float64)
        sig = self._view_f32(sg.value, 1, n.value)[0] if sg.value else None
        return grad, sig

    def tell_end(self) -> None:
        _check(self.lib.evo_tell_end(self._h), "evo_tell_end")

    def capture_generation(self, fitness: torch.Tensor) -> "torch.cuda.CUDAGraph":
        """Captures ask -> rollout -> tell into a CUDA graph; every ``replay()`` is one generation
        (the counters that select the random streams live on the device).  The solver must have
        been created on a non-default stream; the fitness of the last replay is left in ``fitness``."""
        if self.stream.cuda_stream == 0:
            raise ValueError("graph capture needs a solver created with stream=torch.cuda.Stream()")
        assert fitness.dtype == torch.float32 and fitness.is_cuda and fitness.numel() == self.P
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=self.stream):
            self.ask()
            self.rollout(fitness=fitness)
            self.tell(fitness)
        return graph

    def close(self) -> None:
        if getattr(self, "_h", None) is not None:
            self.lib.evo_destroy(self._h)
            self._h = None

    __del__ = close

    # -- helpers -------------------------------------------------------------------------
    def set_batch(self, images: torch.Tensor, labels: torch.Tensor) -> None:
        assert images.dtype == torch.float32 and images.is_cuda and images.is_contiguous()
        assert labels.dtype == torch.int32 and labels.is_cuda and labels.is_contiguous()
        self._batch = (images, labels)           # keep alive
        _check(self.lib.evo_set_batch(self._h, images.data_ptr(), labels.data_ptr()), "evo_set_batch")

    def set_target(self, target: torch.Tensor) -> None:
        """Painting task: the image [H][W][3] (fp32, device) every member's canvas is compared with."""
        assert target.dtype == torch.float32 and target.is_cuda and target.is_contiguous()
        self._target = target                    # keep alive
        _check(self.lib.evo_set_target(self._h, target.data_ptr()), "evo_set_target")

    def padded_rows(self, rows: int) -> torch.Tensor:
        """A zeroed [rows][ldD] device matrix with the pitch evo_rollout expects."""
        return torch.zeros(rows, self.ldD, dtype=torch.float32, device=self.device)

    def _view_f32(self, ptr: int, rows: int, cols: int) -> torch.Tensor:
        off = ptr - self.workspace.data_ptr()
        flat = self.workspace[off:off + rows * cols * 4].view(torch.float32)
        return flat.view(rows, cols)

    def _view_i32(self, ptr: int, n: int) -> torch.Tensor:
        off = ptr - self.workspace.data_ptr()
        return self.workspace[off:off + n * 4].view(torch.int32)

    def center(self) -> torch.Tensor:
        p = C.c_void_p()
        _check(self.lib.evo_get_center(self._h, C.byref(p)), "evo_get_center")
        return self._view_f32(p.value, 1, self.ldD)[0, :self.D]

    def moments(self):
        m, v = C.c_void_p(), C.c_void_p()
        _check(self.lib.evo_get_moments(self._h, C.byref(m), C.byref(v)), "evo_get_moments")
        return (self._view_f32(m.value, 1, self.ldD)[0, :self.D],
                self._view_f32(v.value, 1, self.ldD)[0, :self.D])

    def gradient(self) -> torch.Tensor:
        p = C.c_void_p()
        _check(self.lib.evo_get_gradient(self._h, C.byref(p)), "evo_get_gradient")
        return self._view_f32(p.value, 1, self.ldD)[0, :self.D]

    def ranks(self):
        r, u = C.c_void_p(), C.c_void_p()
        _check(self.lib.evo_get_ranks(self._h, C.byref(r), C.byref(u)), "evo_get_ranks")
        return self._view_i32(r.value, self.P_global), self._view_f32(u.value, 1, self.P_global)[0]

    def eps(self) -> Optional[torch.Tensor]:
        p = C.c_void_p()
        _check(self.lib.evo_get_eps(self._h, C.byref(p)), "evo_get_eps")
        if not p.value:
            return None
        return self._view_f32(p.value, self.P // 2, self.ldD)[:, :self.D]

    def sigma(self) -> torch.Tensor:
        p = C.c_void_p()
        _check(self.lib.evo_get_sigma(self._h, C.byref(p)), "evo_get_sigma")
        return self._view_f32(p.value, 1, self.ldD)[0, :self.D]

    def set_sigma(self, sigma: torch.Tensor) -> None:
        assert sigma.dtype == torch.float32 and sigma.is_cuda and sigma.is_contiguous() and sigma.numel() == self.D
        _check(self.lib.evo_set_sigma(self._h, sigma.data_ptr()), "evo_set_sigma")

    def counters(self):
        g, t = C.c_uint32(), C.c_uint32()
        _check(self.lib.evo_get_counters(self._h, C.byref(g), C.byref(t)), "evo_get_counters")
        return g.value, t.value

    def set_state(self, center=None, m=None, v=None, generation=0, adam_step=0) -> None:
        def ptr(x):
            if x is None:
                return None
            assert x.dtype == torch.float32 and x.is_cuda and x.is_contiguous() and x.numel() == self.D
            return x.data_ptr()
        _check(self.lib.evo_set_state(self._h, ptr(center), ptr(m), ptr(v), generation, adam_step),
               "evo_set_state")

    def debug_check(self):
        """Checked build only: (damaged region or -1, skipped store site or 0, its index)."""
        reg, site, idx = C.c_int32(), C.c_uint32(), C.c_uint64()
        _check(self.lib.evo_debug_check(self._h, C.byref(reg), C.byref(site), C.byref(idx)), "evo_debug_check")
        return reg.value, site.value, idx.value

    def sync_status(self) -> int:
        return self.lib.evo_sync_status(self._h)

    def launch_count(self) -> int:
        n = C.c_uint64()
        _check(self.lib.evo_launch_count(self._h, C.byref(n)), "evo_launch_count")
        return n.value


STATIC_SCRATCH_BYTES = 4 << 20


def es_gradient_static(u: torch.Tensor, eps: torch.Tensor, sigma: float,
                       out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """ES gradient through ``evo_es_gradient_static``: no workspace, no allocation inside the
    library (its scratch is a fixed array in the library image).  ``u`` is [P] fp32, ``eps`` is
    [P/2][D] fp32 with unit column stride (any row pitch); returns g[D].  Meant for hosts that
    forbid device allocation after start-up; pass ``out`` to keep this wrapper allocation-free
    as well.  Calls that may overlap on the GPU must be serialised by the caller."""
    lib = load_library()
    assert u.dtype == torch.float32 and eps.dtype == torch.float32 and u.is_cuda and eps.is_cuda
    assert u.is_contiguous() and eps.stride(1) == 1 and eps.shape[0] * 2 == u.numel()
    P, D = u.numel(), eps.shape[1]
    if out is None:
        out = torch.empty(D, dtype=torch.float32, device=u.device)
    with torch.cuda.device(u.device):
        st = stream if stream is not None else torch.cuda.current_stream(u.device)
        _check(lib.evo_es_gradient_static(u.data_ptr(), eps.data_ptr(), P, D, eps.stride(0), float(sigma),
                                          out.data_ptr(), st.cuda_stream), "evo_es_gradient_static")
    return out
