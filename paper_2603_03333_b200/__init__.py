"""B200 (sm_100a) implementation of the DropMatch MC-dropout LM-head verification step.

The work is done by libdropmatch.so (CUDA, C ABI in include/dropmatch.h); `binding` marshals
torch tensors into it and `workloads` draws seeded synthetic inputs.
"""
from . import binding, workloads  # noqa: F401
from . import vocab_parallel  # noqa: F401
from .binding import Context, DropMatchError  # noqa: F401
