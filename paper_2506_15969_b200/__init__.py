"""B200-native LazyEviction decode hot path: CUDA kernels behind a C ABI.

`paper_2506_15969_b200.binding` loads the shared library and mirrors its entry
points; `paper_2506_15969_b200.traces` generates the seeded synthetic inputs.
Nothing is imported eagerly so that the trace generator can be used without
the CUDA library.
"""
__all__ = ["binding", "traces", "build"]
