"""Seeded synthetic inputs for the five benchmark configurations.

This module only produces INPUTS (sizes, hyper-parameters, per-coordinate
arrays).  It contains none of the method's arithmetic and imports neither the
CUDA binding nor the CPU oracle; both are fed from here so that they see
byte-identical data.

Per-coordinate arrays are generated in fixed chunks of 2**20 coordinates, each
chunk from its own counter-based stream `Philox(key=[seed, chunk])`, so any
coordinate range can be produced without materialising the whole vector (used
for sampled-coordinate parity on the large configurations and for
coordinate-sharded multi-GPU runs).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

CHUNK = 1 << 20
H_NEVER = 0xFFFFFFFF  # "H = +infinity": never synchronise


@dataclass
class Workload:
    name: str
    W: int
    sizes: List[int]            # tensor sizes, packed back to back
    grad: str                   # "noise" | "noise_scaled" | "quadratic"
    eta: float
    eps: float
    H: int
    T: int
    sigma: float = 0.0
    bf16_grads: bool = False
    b0sq: float = 0.0
    noise_seed: int = 0
    array_seed: int = 0
    a_range: Tuple[float, float] = (0.1, 10.0)
    s_range: Tuple[float, float] = (1e-3, 1.0)
    H_sweep: List[int] = field(default_factory=list)

    @property
    def N(self) -> int:
        return int(sum(self.sizes))

    def arrays(self, j0: int = 0, n: Optional[int] = None) -> Dict[str, np.ndarray]:
        """Per-coordinate input arrays for global coordinates [j0, j0+n)."""
        n = self.N - j0 if n is None else n
        out: Dict[str, np.ndarray] = {}
        if self.grad == "quadratic":
            out["a"] = _range_of(self.array_seed, 0, j0, n,
                                 lambda g, m: g.uniform(self.a_range[0], self.a_range[1], m))
            out["c"] = _range_of(self.array_seed, 1, j0, n, lambda g, m: g.standard_normal(m))
        elif self.grad == "noise_scaled":
            lo, hi = np.log(self.s_range[0]), np.log(self.s_range[1])
            out["s"] = _range_of(self.array_seed, 2, j0, n,
                                 lambda g, m: np.exp(g.uniform(lo, hi, m)))
        return out


def _chunk(seed: int, which: int, chunk: int, draw) -> np.ndarray:
    g = np.random.Generator(np.random.Philox(key=[(seed << 8) | which, chunk]))
    return draw(g, CHUNK).astype(np.float32)


def _range_of(seed: int, which: int, j0: int, n: int, draw) -> np.ndarray:
    out = np.empty(n, np.float32)
    first, last = j0 // CHUNK, (j0 + n - 1) // CHUNK if n else j0 // CHUNK - 1

    def fill(ch: int) -> None:
        lo = max(j0, ch * CHUNK)
        hi = min(j0 + n, (ch + 1) * CHUNK)
        out[lo - j0: hi - j0] = _chunk(seed, which, ch, draw)[lo - ch * CHUNK: hi - ch * CHUNK]

    chunks = range(first, last + 1)
    if len(chunks) > 8:      # chunks are independent streams: draw them on several host threads
        import os
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, chunks))
    else:
        for ch in chunks:
            fill(ch)
    return out


def ragged_sizes(count: int = 200, seed: int = 7, total: int = 400_000_000,
                 lo: int = 1024, hi: int = 64 << 20) -> List[int]:
    """`count` tensor sizes, log-uniform on [lo, hi], rescaled to sum to about `total`.

    The raw log-uniform draws sum to roughly three times the requested total, so
    every size is multiplied by total/sum (floored, not below `lo`).
    """
    g = np.random.Generator(np.random.Philox(key=[seed, 0]))
    u = g.uniform(0.0, 1.0, count)
    raw = np.floor(lo * (hi / lo) ** u)
    scaled = np.maximum(np.floor(raw * (total / raw.sum())), lo)
    return [int(v) for v in scaled]


def config(name: str) -> Workload:
    """The five configurations, named c1..c5."""
    if name == "c1":   # tiny correctness case
        return Workload("c1", W=4, sizes=[65536], grad="quadratic", eta=0.1, eps=1.0, H=4, T=64,
                        sigma=0.1, noise_seed=1, array_seed=1001)
    if name == "c2":   # flat tensor, scaled pure noise
        return Workload("c2", W=8, sizes=[1 << 24], grad="noise_scaled", eta=0.01, eps=1e-3, H=8,
                        T=256, noise_seed=2, array_seed=1002)
    if name == "c3":   # language-model-like split into six tensors
        sizes = [1 << 26, 1 << 24, 1 << 24, 1 << 23, 0, 4096]
        sizes[4] = (1 << 27) - sum(sizes)
        return Workload("c3", W=8, sizes=sizes, grad="quadratic", eta=0.2, eps=1.0, H=16, T=64,
                        sigma=1.0, noise_seed=3, array_seed=1003)
    if name == "c4":   # synchronisation-period sweep
        return Workload("c4", W=16, sizes=[1 << 26], grad="noise", eta=0.01, eps=1e-2, H=16, T=256,
                        noise_seed=4, array_seed=1004, H_sweep=[1, 4, 16, 64])
    if name == "c5":   # ragged multi-tensor, bf16-rounded gradients
        return Workload("c5", W=4, sizes=ragged_sizes(), grad="quadratic", eta=0.05, eps=1.0, H=8,
                        T=32, sigma=0.5, bf16_grads=True, noise_seed=5, array_seed=1005,
                        a_range=(0.01, 100.0))
    raise KeyError(name)


def sample_ranges(wl: Workload, span: int = 4096, extra: int = 6, seed: int = 99) -> List[Tuple[int, int]]:
    """Coordinate ranges [j0, j1) for sampled parity: both ends of the vector, a window
    around every tensor boundary, and `extra` seeded random windows.  Starts are
    multiples of 4 (the library's coordinate-group size)."""
    N = wl.N
    want = [(0, min(span, N)), (max(0, (N - span) // 4 * 4), N)]
    off = 0
    for sz in wl.sizes[:-1]:
        off += sz
        lo = max(0, (off - 64) // 4 * 4)
        want.append((lo, min(N, lo + 128)))
    g = np.random.Generator(np.random.Philox(key=[seed, 1]))
    for _ in range(extra):
        lo = int(g.integers(0, max(1, N - span))) // 4 * 4
        want.append((lo, min(N, lo + span)))
    want.sort()
    merged: List[Tuple[int, int]] = []
    for lo, hi in want:
        if merged and lo <= merged[-1][1]:
            merged[-1] = (merged[-1][0], max(merged[-1][1], hi))
        else:
            merged.append((lo, hi))
    return merged
