"""libcott: cosine attention (Cottention) hot path for NVIDIA B200.

Thin Python binding over the C-ABI library ``libcott.so`` (see ``include/cott.h``).
PyTorch is used only to own device memory and streams; every step of the method
runs inside the library's CUDA kernels.  There is no CPU fallback: a missing
library or a missing GPU raises.
"""
from . import cott  # noqa: F401
from .cott import (  # noqa: F401
    CottError, bwd, bwd_stateful, bwd_varlen, decode_step, fwd, fwd_bwd_host, fwd_noalloc, fwd_stateful, fwd_varlen,
    library_path, query_plan, workspace_bytes, workspace_bytes_varlen,
)
