"""G-CADA per-iteration step on one B200 (CUDA kernels behind a C ABI).

`binding` loads the shared library and mirrors its entry points; `workloads`
produces seeded synthetic inputs; `build` compiles the library in-tree.
Nothing is loaded at import time.
"""
__all__ = ["binding", "workloads", "build"]
