"""TEST INFRASTRUCTURE: the fp64 CPU oracle of the routed decode path.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may
import this package.  It shares nothing with the CUDA library.
"""
from .skv_oracle import (Oracle, build_oracle, mu_from_owners, group_map, cache_bytes, count_owners,  # noqa: F401
                         rcla_map, rdcla_map, quantize_e4m3, e4m3_value)
