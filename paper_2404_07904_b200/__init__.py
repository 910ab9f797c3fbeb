"""B200-native HGRN2 recurrence (paper Eq. 3): C-ABI CUDA library plus a thin Python binding.

`binding` marshals torch device tensors into the C ABI declared in ``include/hgrn2.h``;
`workloads` holds the seeded synthetic input recipes; `build` compiles the library in-tree.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]
