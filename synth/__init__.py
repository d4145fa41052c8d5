"""Seeded synthetic inputs: fragment tables of the workloads and the random buffers.

This package holds none of the method's arithmetic.  It only describes *where*
fragments lie in the flat parameter vector and fills buffers with seeded
random numbers.  Both the CPU oracle's tests and the CUDA library's tests and
benchmark draw their inputs from here, so that both sides see identical bits.
"""

from .configs import Workload, Partition, get_workload, WORKLOAD_NAMES, small_workload
from .generate import generate, fragment_scales, DeviceBuffers

__all__ = [
    "Workload", "Partition", "get_workload", "WORKLOAD_NAMES", "small_workload",
    "generate", "fragment_scales", "DeviceBuffers",
]
