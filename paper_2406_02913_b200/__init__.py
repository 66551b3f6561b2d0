"""B200-native hot path of sensitive-sparse zeroth-order fine-tuning (arXiv 2406.02913).

`binding` is the ctypes layer over libszo.so (the C ABI of include/szo.h); `workloads` holds the
seeded synthetic input generators; `build` compiles the CUDA sources with nvcc for sm_100a.
Importing the package loads nothing: the library is opened on first use and its absence is an
error, never a fallback.
"""
__all__ = ["binding", "workloads", "build"]
