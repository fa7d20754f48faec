"""Routed (depth-wise shared) paged KV cache + decode attention for B200.

A thin Python binding over the C-ABI library ``libskv.so`` (see
``include/skv.h``).  Every step of the path runs in the library's CUDA kernels;
this package only marshals arguments.  There is no CPU fallback: importing
:mod:`paper_2604_22782_b200.binding` raises if the library cannot be loaded.
"""
from .binding import (  # noqa: F401
    SkvError, SkvCache, lib, lib_path, exported_symbols,
    skv_routing_from_owners, skv_routing_groups, skv_routing_rcla, skv_routing_rdcla, skv_cache_pool_bytes,
    skv_strerror,
)

__all__ = [
    "SkvError", "SkvCache", "lib", "lib_path", "exported_symbols",
    "skv_routing_from_owners", "skv_routing_groups", "skv_routing_rcla", "skv_routing_rdcla",
    "skv_cache_pool_bytes", "skv_strerror",
]
