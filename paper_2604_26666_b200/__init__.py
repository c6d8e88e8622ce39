"""libfact for B200: fused-epilogue BF16 GEMMs as hand-written sm_100a kernels.

``binding`` is the ctypes layer over the C ABI of ``include/fact.h``;
``workloads`` names the benchmark shapes and draws their seeded inputs;
``build`` compiles ``libfact.so`` in-tree.  Importing the package does not
load the library; the first ``Handle`` does, and raises if it is missing.
"""
from .binding import Config, FactError, Handle, lib  # noqa: F401
