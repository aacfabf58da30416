"""Sparse MoE feed-forward layer (CoSMoEs, arXiv 2503.00245) on B200: sm_100a kernels behind a C ABI.

`binding` mirrors include/cosmoe.h; `layer` adds the small conveniences (packing weights, owning
a context and its workspace) that callers and the benchmark use.
"""
from . import binding  # noqa: F401
from .layer import MoELayer, OffloadedStack, pack_dense, pack_wd  # noqa: F401
