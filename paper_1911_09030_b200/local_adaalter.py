"""ctypes binding of the C-ABI in `include/local_adaalter.h` — same names, argument
marshalling only.  Every step of Algorithm 3 (Local AdaAlter) runs in the CUDA kernels of
`liblocal_adaalter.so`; PyTorch is used for device memory (the state arena) and streams.

There is no CPU fallback: if the shared library is missing the import of `lib()` raises.
Build it with `python -m paper_1911_09030_b200.build`.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# LA_LIBRARY=debug selects the checked build (same code compiled with -DLA_DEBUG: every kernel
# address is range-checked and violations surface as LA_EBOUNDS at the next synchronising call).
LIB_PATH = os.path.join(_HERE, "liblocal_adaalter_debug.so" if os.environ.get("LA_LIBRARY") == "debug"
                        else "liblocal_adaalter.so")

LA_OK, LA_EINVAL, LA_ENOMEM, LA_ECUDA, LA_ESTATE, LA_ETOOBIG, LA_EBOUNDS = 0, -1, -2, -3, -4, -5, -6
LA_STATIC_SCRATCH_MAX_COORDS = 1048576
LA_F32, LA_BF16 = 0, 1
LA_FUSE_NONE, LA_FUSE_STEP_SYNC, LA_FUSE_SYNC_STEP, LA_FUSE_PERIOD, LA_FUSE_MEAN_ONCE = 0, 1, 2, 3, 4
LA_RULE_ADAALTER, LA_RULE_LOCAL_SGD, LA_RULE_ADAGRAD = 0, 1, 2
LA_H_NEVER = 0xFFFFFFFF
LA_MAX_WORKERS = 64


class la_config(C.Structure):
    _fields_ = [("K", C.c_uint32), ("sizes", C.POINTER(C.c_uint64)), ("j_base", C.c_uint64),
                ("W", C.c_uint32), ("H", C.c_uint32), ("eta", C.c_float), ("eps", C.c_float),
                ("b0sq", C.c_float), ("dev_arena", C.c_void_p), ("arena_bytes", C.c_uint64),
                ("stream", C.c_void_p), ("device", C.c_int32)]


class la_stats(C.Structure):
    _fields_ = [("launches_local", C.c_uint64), ("launches_sync", C.c_uint64),
                ("launches_fused", C.c_uint64), ("launches_other", C.c_uint64),
                ("ms_local", C.c_double), ("ms_sync", C.c_double), ("ms_fused", C.c_double),
                ("bytes_local", C.c_double), ("bytes_sync", C.c_double), ("bytes_fused", C.c_double),
                ("launches_step_sync", C.c_uint64), ("launches_sync_step", C.c_uint64),
                ("launches_period", C.c_uint64),
                ("ms_step_sync", C.c_double), ("ms_sync_step", C.c_double), ("ms_period", C.c_double),
                ("bytes_step_sync", C.c_double), ("bytes_sync_step", C.c_double), ("bytes_period", C.c_double)]


class la_stream_io(C.Structure):
    _fields_ = [("x0_host", C.c_void_p), ("a_host", C.c_void_p), ("c_host", C.c_void_p), ("s_host", C.c_void_p),
                ("worker", C.c_uint32), ("x_host", C.c_void_p), ("b2_host", C.c_void_p), ("bs_host", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Load the CUDA library; raise if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: run `python -m paper_1911_09030_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, u64, u32, f32, i32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_float, C.c_int
        pp = C.POINTER(vp)
        sig = {
            "la_create": [pp, u64, u32, f32, f32, u32],
            "la_create_ex": [pp, C.POINTER(la_config)],
            "la_arena_bytes": [C.POINTER(la_config), C.POINTER(u64)],
            "la_set_init": [vp, vp, f32],
            "la_set_grad_noise": [vp, u64, vp],
            "la_set_grad_quadratic": [vp, u64, vp, vp, f32],
            "la_set_grad_constant": [vp, vp],
            "la_set_grad_dtype": [vp, i32],
            "la_set_identical_workers": [vp, i32],
            "la_set_warmup": [vp, u32],
            "la_set_fusion": [vp, i32],
            "la_set_rule": [vp, i32],
            "la_set_launch_shape": [vp, i32],
            "la_set_profiling": [vp, i32],
            "la_set_graph": [vp, i32],
            "la_local_step": [vp],
            "la_local_step_grads": [vp, vp, i32],
            "la_step_grads": [vp, vp, i32],
            "la_sync": [vp],
            "la_run": [vp, u64],
            "la_read_state": [vp, u32, vp, vp, vp],
            "la_write_state": [vp, u32, vp, vp, vp],
            "la_read_range": [vp, u32, u64, u64, vp, vp, vp],
            "la_tensor_range": [vp, u32, C.POINTER(u64), C.POINTER(u64)],
            "la_get_counters": [vp, C.POINTER(u64), C.POINTER(u32), C.POINTER(u64)],
            "la_set_counters": [vp, u64, u32, u64],
            "la_get_stats": [vp, C.POINTER(la_stats), i32],
            "la_diagnostics": [vp, C.POINTER(C.c_double), C.POINTER(C.c_double)],
            "la_set_worker_range": [vp, u32, u32],
            "la_comm_create": [vp, u32, u32],
            "la_comm_buffer": [vp, C.POINTER(vp), C.POINTER(u64)],
            "la_comm_ipc_handle": [vp, vp],
            "la_comm_open_peer": [vp, u32, vp],
            "la_comm_set_peer": [vp, u32, vp],
            "la_comm_export": [vp],
            "la_comm_combine": [vp],
            "la_comm_import": [vp],
            "la_comm_step_export": [vp],
            "la_comm_step_grads_export": [vp, vp, i32],
            "la_comm_import_step": [vp],
            "la_comm_import_step_grads": [vp, vp, i32],
            "la_stream_sync": [vp],
            "la_noise_tables": [vp, vp, vp, vp],
            "la_replica_means_static": [vp, vp, u32, u64, u64, vp, vp, vp],
            "la_run_streamed": [vp, u64, C.POINTER(la_stream_io), u32],
            "la_debug_build": [],
            "la_debug_narrow": [vp, u64],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.la_destroy.argtypes = [vp]
        L.la_destroy.restype = None
        L.la_last_error.argtypes = [vp]
        L.la_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def replica_means_static(x_ptr, b2_ptr, W, n, stride, x_mean_ptr, b2_mean_ptr, stream=None) -> int:
    """`la_replica_means_static`: replica average without any allocation (for callers whose device
    memory is all spoken for).  Arguments are raw device addresses; returns the status code."""
    return lib().la_replica_means_static(C.c_void_p(int(x_ptr)), C.c_void_p(int(b2_ptr)), int(W), int(n), int(stride),
                                         C.c_void_p(int(x_mean_ptr)), C.c_void_p(int(b2_mean_ptr)),
                                         C.c_void_p(int(stream)) if stream else None)


def debug_build() -> bool:
    """True when the loaded library is the checked build."""
    return bool(lib().la_debug_build())


def noise_tables(radius_ptr=None, cos_ptr=None, sin_ptr=None, stream=None) -> int:
    """`la_noise_tables`: fill device buffers of 2^24 floats each (raw addresses, None to skip)."""
    vp = lambda p: C.c_void_p(int(p)) if p else None
    return lib().la_noise_tables(vp(radius_ptr), vp(cos_ptr), vp(sin_ptr), vp(stream))


class LocalAdaAlterError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"[{code}] {msg}")
        self.code = code


def _hostptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _as_f32(a, n, what):
    """Accept a numpy array or a CPU torch tensor (e.g. pinned) of n float32 values."""
    if a is None:
        return None, None
    if hasattr(a, "data_ptr"):                     # torch tensor on the host
        if a.device.type != "cpu" or str(a.dtype) != "torch.float32" or not a.is_contiguous() or a.numel() != n:
            raise ValueError(f"{what}: need a contiguous CPU float32 tensor of {n} elements")
        return a, C.c_void_p(a.data_ptr())
    arr = np.ascontiguousarray(a, dtype=np.float32)
    if arr.shape != (n,):
        raise ValueError(f"{what}: need {n} float32 values, got shape {arr.shape}")
    return arr, _hostptr(arr)


class LocalAdaAlter:
    """Handle around one `la_ctx`.  Method names mirror the C functions without the prefix."""

    def __init__(self, sizes: Sequence[int] | int, W: int, eta: float, eps: float, H: int,
                 b0sq: float = 0.0, j_base: int = 0, stream: Optional[int] = None,
                 device: int = -1, arena=None):
        self.L = lib()
        sizes = [int(sizes)] if np.isscalar(sizes) else [int(s) for s in sizes]
        self.sizes = sizes
        self.N = sum(sizes)
        self.W = int(W)
        self._sizes_arr = (C.c_uint64 * len(sizes))(*sizes)
        cfg = la_config()
        cfg.K = len(sizes)
        cfg.sizes = C.cast(self._sizes_arr, C.POINTER(C.c_uint64))
        cfg.j_base = int(j_base)
        cfg.W, cfg.H, cfg.eta, cfg.eps, cfg.b0sq = int(W), int(H), float(eta), float(eps), float(b0sq)
        cfg.stream = C.c_void_p(stream) if stream else None
        cfg.device = int(device)
        self._arena = arena                         # keep the torch tensor alive
        if arena is not None:
            cfg.dev_arena = C.c_void_p(arena.data_ptr())
            cfg.arena_bytes = arena.numel() * arena.element_size()
        self.h = C.c_void_p()
        rc = self.L.la_create_ex(C.byref(self.h), C.byref(cfg))
        if rc != LA_OK:
            self.h = None
            raise LocalAdaAlterError(rc, self.L.la_last_error(None).decode())

    @staticmethod
    def arena_bytes(sizes: Sequence[int], W: int, eta=0.1, eps=1.0, H=1) -> int:
        L = lib()
        arr = (C.c_uint64 * len(sizes))(*[int(s) for s in sizes])
        cfg = la_config()
        cfg.K = len(sizes)
        cfg.sizes = C.cast(arr, C.POINTER(C.c_uint64))
        cfg.W, cfg.H, cfg.eta, cfg.eps = int(W), int(H), float(eta), float(eps)
        out = C.c_uint64()
        rc = L.la_arena_bytes(C.byref(cfg), C.byref(out))
        if rc != LA_OK:
            raise LocalAdaAlterError(rc, L.la_last_error(None).decode())
        return out.value

    @classmethod
    def with_torch_arena(cls, sizes, W, eta, eps, H, **kw):
        """State memory from PyTorch's allocator, kernels on PyTorch's current stream."""
        import torch
        sizes = [int(sizes)] if np.isscalar(sizes) else [int(s) for s in sizes]
        nbytes = cls.arena_bytes(sizes, W, eta, eps, H)
        arena = torch.empty(nbytes // 4, dtype=torch.float32, device="cuda")
        stream = torch.cuda.current_stream().cuda_stream
        return cls(sizes, W, eta, eps, H, stream=stream, arena=arena,
                   device=torch.cuda.current_device(), **kw)

    # ------------------------------------------------------------------ plumbing
    def _ck(self, rc):
        if rc != LA_OK:
            raise LocalAdaAlterError(rc, self.L.la_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.L.la_destroy(self.h)
            self.h = None

    destroy = close

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ configuration
    def set_init(self, x0=None, b0sq=0.0):
        keep, p = _as_f32(x0, self.N, "x0")
        self._ck(self.L.la_set_init(self.h, p, float(b0sq)))
        self.sync_stream() if keep is not None else None

    def set_grad_noise(self, seed, s=None):
        keep, p = _as_f32(s, self.N, "s")
        self._ck(self.L.la_set_grad_noise(self.h, int(seed), p))
        self.sync_stream() if keep is not None else None

    def set_grad_quadratic(self, seed, a, c, sigma):
        ka, pa = _as_f32(a, self.N, "a")
        kc, pc = _as_f32(c, self.N, "c")
        self._ck(self.L.la_set_grad_quadratic(self.h, int(seed), pa, pc, float(sigma)))
        self.sync_stream()

    def set_grad_constant(self, s=None):
        keep, p = _as_f32(s, self.N, "s")
        self._ck(self.L.la_set_grad_constant(self.h, p))
        self.sync_stream() if keep is not None else None

    def set_grad_dtype(self, dtype):
        self._ck(self.L.la_set_grad_dtype(self.h, int(dtype)))

    def set_identical_workers(self, on=True):
        self._ck(self.L.la_set_identical_workers(self.h, int(bool(on))))

    def set_warmup(self, steps):
        self._ck(self.L.la_set_warmup(self.h, int(steps)))

    def set_rule(self, rule):
        self._ck(self.L.la_set_rule(self.h, int(rule)))

    def set_fusion(self, mode):
        self._ck(self.L.la_set_fusion(self.h, int(mode)))

    def set_launch_shape(self, blocks_per_sm):
        self._ck(self.L.la_set_launch_shape(self.h, int(blocks_per_sm)))

    def set_graph(self, on=True):
        self._ck(self.L.la_set_graph(self.h, int(bool(on))))

    def set_profiling(self, on=True):
        self._ck(self.L.la_set_profiling(self.h, int(bool(on))))

    # ------------------------------------------------------------------ hot path
    def local_step(self):
        self._ck(self.L.la_local_step(self.h))

    def local_step_grads(self, g_dev_ptr: int, dtype=LA_F32):
        self._ck(self.L.la_local_step_grads(self.h, C.c_void_p(int(g_dev_ptr)), int(dtype)))

    def step_grads(self, g_dev_ptr: int, dtype=LA_F32):
        self._ck(self.L.la_step_grads(self.h, C.c_void_p(int(g_dev_ptr)), int(dtype)))

    def sync(self):
        self._ck(self.L.la_sync(self.h))

    def run(self, T):
        self._ck(self.L.la_run(self.h, int(T)))

    def run_streamed(self, T, worker=0, x0=None, a=None, c=None, s=None, x_out=None, b2_out=None, bs_out=None,
                     chunks=0):
        """`la_run_streamed`: init from host arrays, T iterations, read-back of one worker — pipelined
        over coordinate ranges.  Arrays are float32 numpy arrays or CPU torch tensors (pinned for overlap)
        of N elements; outputs are written in place."""
        keep, io = [], la_stream_io()
        for name, arr in (("x0_host", x0), ("a_host", a), ("c_host", c), ("s_host", s),
                          ("x_host", x_out), ("b2_host", b2_out), ("bs_host", bs_out)):
            k, ptr = _as_f32(arr, self.N, name)
            if arr is not None and name in ("x_host", "b2_host", "bs_host") and k is not arr:
                raise ValueError(f"{name}: outputs must be contiguous float32 buffers of {self.N} elements")
            keep.append(k)
            setattr(io, name, ptr.value if ptr is not None else None)
        io.worker = int(worker)
        self._ck(self.L.la_run_streamed(self.h, int(T), C.byref(io), int(chunks)))

    # ------------------------------------------------------------------ state
    def read_state(self, worker, want=("x", "b2", "bs"), out=None):
        """Returns (x, b2, bs) as numpy arrays (None for the ones not requested)."""
        bufs = {}
        for k in ("x", "b2", "bs"):
            if k in want:
                bufs[k] = out[k] if out and k in out else np.empty(self.N, np.float32)
        ptr = lambda k: (C.c_void_p(bufs[k].data_ptr()) if hasattr(bufs.get(k), "data_ptr")
                         else _hostptr(bufs.get(k)))
        self._ck(self.L.la_read_state(self.h, int(worker), ptr("x"), ptr("b2"), ptr("bs")))
        return bufs.get("x"), bufs.get("b2"), bufs.get("bs")

    def read_range(self, worker, j0, n):
        x, b2, bs = (np.empty(n, np.float32) for _ in range(3))
        self._ck(self.L.la_read_range(self.h, int(worker), int(j0), int(n), _hostptr(x), _hostptr(b2), _hostptr(bs)))
        return x, b2, bs

    def write_state(self, worker, x=None, b2=None, bs=None):
        kx, px = _as_f32(x, self.N, "x")
        kb, pb = _as_f32(b2, self.N, "b2")
        ks, ps = _as_f32(bs, self.N, "bs")
        self._ck(self.L.la_write_state(self.h, int(worker), px, pb, ps))

    def tensor_range(self, k):
        off, sz = C.c_uint64(), C.c_uint64()
        self._ck(self.L.la_tensor_range(self.h, int(k), C.byref(off), C.byref(sz)))
        return off.value, sz.value

    def get_counters(self):
        t, tp, ns = C.c_uint64(), C.c_uint32(), C.c_uint64()
        self._ck(self.L.la_get_counters(self.h, C.byref(t), C.byref(tp), C.byref(ns)))
        return t.value, tp.value, ns.value

    def set_counters(self, t, tp, nsync):
        self._ck(self.L.la_set_counters(self.h, int(t), int(tp), int(nsync)))

    def get_stats(self, reset=False):
        st = la_stats()
        self._ck(self.L.la_get_stats(self.h, C.byref(st), int(bool(reset))))
        return {k: getattr(st, k) for k, _ in la_stats._fields_}

    def diagnostics(self):
        """(objective at the mean iterate, mean squared distance of the replicas from it)."""
        f, d = C.c_double(), C.c_double()
        self._ck(self.L.la_diagnostics(self.h, C.byref(f), C.byref(d)))
        return f.value, d.value

    def debug_narrow(self, nbytes):
        """Checked build only: treat the last `nbytes` bytes of the arena as foreign (0 restores)."""
        self._ck(self.L.la_debug_narrow(self.h, int(nbytes)))

    def sync_stream(self):
        """Block until the context's stream is idle."""
        self._ck(self.L.la_stream_sync(self.h))

    stream_sync = sync_stream

    # ------------------------------------------------------------------ sharding by worker
    def set_worker_range(self, worker_base, W_total):
        self._ck(self.L.la_set_worker_range(self.h, int(worker_base), int(W_total)))

    def comm_create(self, rank, world):
        self._ck(self.L.la_comm_create(self.h, int(rank), int(world)))

    def comm_buffer(self):
        """(device pointer, bytes) of the exchange buffer."""
        p, n = C.c_void_p(), C.c_uint64()
        self._ck(self.L.la_comm_buffer(self.h, C.byref(p), C.byref(n)))
        return p.value, n.value

    def comm_ipc_handle(self) -> bytes:
        buf = C.create_string_buffer(64)
        self._ck(self.L.la_comm_ipc_handle(self.h, buf))
        return buf.raw

    def comm_open_peer(self, peer_rank, handle: bytes):
        buf = C.create_string_buffer(handle, 64)
        self._ck(self.L.la_comm_open_peer(self.h, int(peer_rank), buf))

    def comm_set_peer(self, peer_rank, dev_ptr):
        self._ck(self.L.la_comm_set_peer(self.h, int(peer_rank), C.c_void_p(int(dev_ptr))))

    def comm_export(self):
        self._ck(self.L.la_comm_export(self.h))

    def comm_combine(self):
        self._ck(self.L.la_comm_combine(self.h))

    def comm_import(self):
        self._ck(self.L.la_comm_import(self.h))

    def comm_step_export(self):
        self._ck(self.L.la_comm_step_export(self.h))

    def comm_step_grads_export(self, g_dev_ptr, dtype=LA_F32):
        self._ck(self.L.la_comm_step_grads_export(self.h, C.c_void_p(int(g_dev_ptr)), int(dtype)))

    def comm_import_step(self):
        self._ck(self.L.la_comm_import_step(self.h))

    def comm_import_step_grads(self, g_dev_ptr, dtype=LA_F32):
        self._ck(self.L.la_comm_import_step_grads(self.h, C.c_void_p(int(g_dev_ptr)), int(dtype)))
