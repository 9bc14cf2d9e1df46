"""B200 (sm_100a) Conv2d -> BatchNorm(batch statistics) -> SiLU block, forward and backward, behind a C ABI.

``binding`` mirrors include/nb_cbs.h through ctypes; ``block`` holds device buffers for one block;
``workloads`` names the detector's layer shapes and draws seeded synthetic inputs; ``build`` compiles the
CUDA library.  Importing the package does not load the library; the first call through ``binding`` does,
and raises if it is missing.
"""
__all__ = ["binding", "block", "workloads", "build"]
