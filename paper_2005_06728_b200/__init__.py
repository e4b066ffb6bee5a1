"""OD-SGD parameter-update pass for NVIDIA B200: CUDA library + thin binding.

`binding` wraps the C ABI of libodsgd.so (include/odsgd.h); `workloads` holds the
seeded synthetic parameter sets; `build` compiles the library in-tree.
"""
__all__ = ["binding", "workloads", "build"]
