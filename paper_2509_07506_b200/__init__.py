"""B200 (sm_100a) kernels for fused_add_rmsnorm, silu_and_mul and merge_attn_states_lse.

``binding`` holds the Python side of the C ABI declared in ``include/astra.h``; ``workloads`` the
seeded synthetic inputs; ``build`` compiles the shared library.  Importing the package does not
load the library; the first call does, and fails loudly if it has not been built.
"""
from .graphs import CapturedCalls  # noqa: F401
from .binding import (  # noqa: F401
    AstraError,
    PreparedCall,
    astra_fused_add_rmsnorm,
    astra_fused_allreduce_add_rmsnorm,
    astra_fused_allreduce_add_rmsnorm_ex,
    prepare_fused_add_rmsnorm,
    prepare_fused_allreduce_add_rmsnorm,
    prepare_merge_attn_states_lse,
    prepare_silu_and_mul,
    astra_fused_add_rmsnorm_ex,
    astra_merge_attn_states_lse,
    astra_merge_attn_states_lse_ex,
    astra_silu_and_mul,
    astra_silu_and_mul_ex,
    load_library,
    status_string,
)
