"""okq: 2-bit KV-cache quantisation and fused decode attention for B200 (sm_100a).

The product is the C-ABI library `libokq.so` (see include/okq.h); `binding` marshals
arguments to it, `workloads` draws seeded synthetic inputs, `build` compiles the library.
"""
from . import workloads  # noqa: F401
