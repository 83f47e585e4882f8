"""B200-native chunk attention over a paged KV cache (HAT cloud-side hot path).

`workloads` draws seeded synthetic inputs; `binding` is the thin ctypes layer over
the C-ABI library built from `csrc/`.  Importing the package loads no native code;
`binding` raises if the CUDA library is missing when first used.
"""
__all__ = ["workloads", "binding", "build"]
