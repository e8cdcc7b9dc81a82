"""ctypes front end of the C++ oracle (`local_adaalter_oracle.cpp`).

TEST INFRASTRUCTURE ONLY: a thin handle class around the plain single-threaded
C++ restatement of Algorithm 3 (Local AdaAlter).  It holds no arithmetic of its
own; every number comes from the C++ file next to it.  The shared object is
compiled on first use with the host compiler (`g++ -O2 -ffp-contract=off`), so
every fp32 line of the C++ source is exactly one IEEE operation.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "local_adaalter_oracle.cpp")
_LIB = os.path.join(_HERE, "liblocal_adaalter_oracle.so")
_lock = threading.Lock()
_lib = None


def _has_fma() -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            return " fma " in f.read().replace("\n", " ")
    except OSError:
        return False


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", _LIB + ".tmp", _SRC]
    if _has_fma():
        cmd.insert(5, "-mfma")  # hardware fmaf; the result is the same either way
    subprocess.run(cmd, check=True)
    os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            # LA_ORACLE_SO: load a pre-built (e.g. deliberately mutated) oracle instead;
            # used only by the mutation test that checks the pins have teeth.
            L = C.CDLL(os.environ.get("LA_ORACLE_SO") or build())
            u64, u32, f32, vp = C.c_uint64, C.c_uint32, C.c_float, C.c_void_p
            L.ora_create.restype = vp
            L.ora_create.argtypes = [u64, u64, u32, f32, f32, u32, f32, vp]
            L.ora_destroy.argtypes = [vp]
            L.ora_set_grad_noise.argtypes = [vp, u64, vp]
            L.ora_set_grad_quadratic.argtypes = [vp, u64, vp, vp, f32]
            L.ora_set_grad_constant.argtypes = [vp, vp]
            L.ora_set_grad_bf16.argtypes = [vp, C.c_int]
            L.ora_set_identical_workers.argtypes = [vp, C.c_int]
            L.ora_set_warmup.argtypes = [vp, u32]
            L.ora_set_rule.argtypes = [vp, C.c_int]
            L.ora_set_worker_base.argtypes = [vp, u32]
            L.ora_local_step.argtypes = [vp]
            L.ora_local_step_grads.argtypes = [vp, vp]
            L.ora_sync.argtypes = [vp]
            L.ora_run.argtypes = [vp, u64]
            L.ora_read.argtypes = [vp, u32, vp, vp, vp]
            L.ora_read_shadow.argtypes = [vp, u32, vp, vp, vp]
            L.ora_write.argtypes = [vp, u32, vp, vp, vp]
            L.ora_get_counters.argtypes = [vp, vp, vp, vp]
            L.ora_set_counters.argtypes = [vp, u64, u32, u64]
            L.ora_mix64.restype = u64
            L.ora_mix64.argtypes = [u64]
            L.ora_stream_key.restype = u64
            L.ora_stream_key.argtypes = [u64, u64, u32]
            L.ora_neg2ln_u24.restype = f32
            L.ora_neg2ln_u24.argtypes = [u32]
            L.ora_cossin_u24.argtypes = [u32, vp, vp]
            L.ora_bf16_round.restype = f32
            L.ora_bf16_round.argtypes = [f32]
            L.ora_noise_fill.argtypes = [u64, u64, u32, u64, u64, vp]
            L.ora_uniform_bits.argtypes = [u64, u64, u32, u64, vp, vp]
            L.ora_scan_neg2ln.argtypes = [vp]
            L.ora_scan_cossin.argtypes = [vp]
            L.ora_table_neg2ln.argtypes = [vp]
            L.ora_table_cossin.argtypes = [vp, vp]
            _lib = L
    return _lib


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Oracle:
    """One simulated job: W workers over `n` coordinates starting at global index `j_base`."""

    def __init__(self, n, W, eta, eps, H, b0sq=0.0, x0=None, j_base=0):
        self.L = lib()
        self.n, self.W, self.H = int(n), int(W), int(H)
        x0 = _f32(x0)
        if x0 is not None and x0.shape != (self.n,):
            raise ValueError("x0 must have n elements")
        self.h = self.L.ora_create(self.n, int(j_base), self.W, float(eta), float(eps),
                                   self.H, float(b0sq), _ptr(x0))
        if not self.h:
            raise ValueError("invalid oracle configuration")

    def close(self):
        if getattr(self, "h", None):
            self.L.ora_destroy(self.h)
            self.h = None

    __del__ = close

    # ---- gradient source -------------------------------------------------
    def set_grad_noise(self, seed, s=None):
        s = _f32(s)
        assert s is None or s.shape == (self.n,)
        self.L.ora_set_grad_noise(self.h, int(seed), _ptr(s))

    def set_grad_quadratic(self, seed, a, c, sigma):
        a, c = _f32(a), _f32(c)
        assert a.shape == (self.n,) and c.shape == (self.n,)
        self.L.ora_set_grad_quadratic(self.h, int(seed), _ptr(a), _ptr(c), float(sigma))

    def set_grad_constant(self, s=None):
        s = _f32(s)
        assert s is None or s.shape == (self.n,)
        self.L.ora_set_grad_constant(self.h, _ptr(s))

    def set_grad_bf16(self, on=True):
        self.L.ora_set_grad_bf16(self.h, int(bool(on)))

    def set_identical_workers(self, on=True):
        self.L.ora_set_identical_workers(self.h, int(bool(on)))

    def set_warmup(self, steps):
        self.L.ora_set_warmup(self.h, int(steps))

    def set_worker_base(self, base):
        """Noise of local worker i is that of global worker base + i."""
        self.L.ora_set_worker_base(self.h, int(base))

    def set_rule(self, rule):
        """0 = Local AdaAlter (Algorithm 3), 1 = Local SGD (Algorithm 2), 2 = Distributed AdaGrad (Algorithm 1)."""
        self.L.ora_set_rule(self.h, int(rule))

    # ---- schedule ----------------------------------------------------------
    def local_step(self, grads=None):
        if grads is None:
            self.L.ora_local_step(self.h)
        else:
            g = _f32(grads)
            assert g.shape == (self.W, self.n)
            self.L.ora_local_step_grads(self.h, _ptr(g))

    def sync(self):
        self.L.ora_sync(self.h)

    def run(self, T):
        self.L.ora_run(self.h, int(T))

    # ---- state ---------------------------------------------------------------
    def read(self, worker):
        x = np.empty(self.n, np.float32)
        b2 = np.empty(self.n, np.float32)
        bs = np.empty(self.n, np.float32)
        self.L.ora_read(self.h, int(worker), _ptr(x), _ptr(b2), _ptr(bs))
        return x, b2, bs

    def read_shadow(self, worker):
        x = np.empty(self.n, np.float64)
        b2 = np.empty(self.n, np.float64)
        bs = np.empty(self.n, np.float64)
        self.L.ora_read_shadow(self.h, int(worker), _ptr(x), _ptr(b2), _ptr(bs))
        return x, b2, bs

    def read_all(self):
        xs, bs2 = [], []
        for i in range(self.W):
            x, b2, bs = self.read(i)
            xs.append(x)
            bs2.append(b2)
        return np.stack(xs), np.stack(bs2), bs

    def write(self, worker, x=None, b2=None, bs=None):
        x, b2, bs = _f32(x), _f32(b2), _f32(bs)
        self.L.ora_write(self.h, int(worker), _ptr(x), _ptr(b2), _ptr(bs))

    def counters(self):
        t, tp, ns = C.c_uint64(), C.c_uint32(), C.c_uint64()
        self.L.ora_get_counters(self.h, C.byref(t), C.byref(tp), C.byref(ns))
        return t.value, tp.value, ns.value

    def set_counters(self, t, tp, nsync):
        self.L.ora_set_counters(self.h, int(t), int(tp), int(nsync))


# ---- gradient-source primitives (for the pins) -----------------------------
def mix64(z):
    return lib().ora_mix64(z & 0xFFFFFFFFFFFFFFFF)


def stream_key(seed, t, worker):
    return lib().ora_stream_key(int(seed), int(t), int(worker))


def neg2ln_u24(k):
    return float(lib().ora_neg2ln_u24(int(k)))


def cossin_u24(q):
    c, s = C.c_float(), C.c_float()
    lib().ora_cossin_u24(int(q), C.byref(c), C.byref(s))
    return c.value, s.value


def bf16_round(g):
    return float(lib().ora_bf16_round(float(g)))


def noise_fill(seed, t, worker, j0, n):
    out = np.empty(int(n), np.float32)
    lib().ora_noise_fill(int(seed), int(t), int(worker), int(j0), int(n), _ptr(out))
    return out


def uniform_bits(seed, t, worker, p):
    k, q = C.c_uint32(), C.c_uint32()
    lib().ora_uniform_bits(int(seed), int(t), int(worker), int(p), C.byref(k), C.byref(q))
    return k.value, q.value


def scan_neg2ln():
    out = np.zeros(4, np.float64)
    lib().ora_scan_neg2ln(_ptr(out))
    return dict(max_abs=out[0], max_rel=out[1], min_L=out[2], L_at_one=out[3])


def table_neg2ln():
    """L[k-1] = -2 ln(k 2^-24) by the recipe, for every k in 1..2^24."""
    out = np.empty(1 << 24, np.float32)
    lib().ora_table_neg2ln(_ptr(out))
    return out


def table_cossin():
    """(cos, sin)(2 pi q 2^-24) by the recipe, for every q in 0..2^24-1."""
    c, s = np.empty(1 << 24, np.float32), np.empty(1 << 24, np.float32)
    lib().ora_table_cossin(_ptr(c), _ptr(s))
    return c, s


def scan_cossin():
    out = np.zeros(3, np.float64)
    lib().ora_scan_cossin(_ptr(out))
    return dict(max_cos=out[0], max_sin=out[1], max_norm=out[2])
