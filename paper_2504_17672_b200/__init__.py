"""CoCoDC outer synchronisation step for NVIDIA B200: Python binding of the C-ABI CUDA library.

The binding only marshals arguments (tensor addresses, sizes, the current CUDA
stream) into the `cocodc_*` entry points of libcocodc.so; every step of the
method runs in that library's kernels.  There is no fallback: if the library is
missing or does not load, importing `paper_2504_17672_b200.binding` raises.
"""

__all__ = ["binding", "build"]
