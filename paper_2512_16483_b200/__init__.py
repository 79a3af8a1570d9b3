"""B200-native late-scale step of VAR next-scale prediction under FasterVAR.

`binding` is the ctypes layer over the C-ABI library libfvar.so (include/fvar.h); `schedule`
holds the host-side rank / stage schedule; `build` compiles the library with nvcc for sm_100a.
Nothing here imports the CPU oracle and nothing falls back to the CPU.
"""
from . import schedule  # noqa: F401

__all__ = ["binding", "schedule", "build"]
