"""SureLock locked-forward hot path for NVIDIA B200 (sm_100a).

`paper_2602_06412_b200.binding` is the thin ctypes layer over the C-ABI library
built from `csrc/`; `paper_2602_06412_b200.inputs` draws the seeded synthetic
workloads.  Importing the package loads nothing native; `binding.lib()` does, and
raises if the library has not been built.
"""

__all__ = ["binding", "inputs", "build"]
