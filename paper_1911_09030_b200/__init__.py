"""B200-native hot path of Local AdaAlter (arXiv 1911.09030, Algorithm 3).

`local_adaalter` is the thin ctypes binding over the C-ABI library
(`include/local_adaalter.h`); `workloads` holds the seeded synthetic inputs.
"""
__all__ = ["workloads", "local_adaalter"]
