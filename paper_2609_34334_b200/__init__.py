"""B200-native zero-SM ring collectives (HOCCL's data-parallel hot path, one GPU, R logical ranks).

`workloads` holds the seeded input generators and workload shapes; `binding` is the thin ctypes
layer over the C-ABI library `libhoccl.so` built from `csrc/` (see `build.py`).  Importing the
package loads nothing; the library is loaded on first use of `binding`.
"""
__all__ = ["workloads", "binding", "build"]
