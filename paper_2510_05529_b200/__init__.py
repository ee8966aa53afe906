"""H1B-KV decode attention over a hybrid 1-bit-key / 4-bit-value cache, CUDA (sm_100a).

The product is the C-ABI library declared in include/h1b.h (built in-tree as
libh1b.so by `paper_2510_05529_b200.build`); `binding` is its ctypes wrapper.
"""
from .build import LIB_PATH, build_library  # noqa: F401

__all__ = ["LIB_PATH", "build_library"]
