"""B200-native transfer dock: put/get dispatch of GRPO samples in HBM.

`paper_2507_19017_b200.binding` is the thin ctypes layer over the C-ABI library
declared in include/td.h; `paper_2507_19017_b200.workloads` draws the seeded
synthetic inputs.  Importing the package loads neither torch nor the library.
"""
__all__ = ["binding", "workloads", "build"]
