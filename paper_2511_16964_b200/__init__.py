"""B200-native fused operator chains (GEMM + epilogue + row reduction, MLP block,
causal attention) behind a C ABI; this package is the thin Python binding."""
from .binding import (  # noqa: F401
    PikeError,
    library_path,
    load_library,
    pike_attention_chain,
    pike_attention_chain_workspace,
    pike_get_last_device_status,
    pike_linear_epilogue,
    pike_linear_epilogue_workspace,
    pike_linear_softmax_noalloc,
    pike_mlp_block,
    pike_mlp_block_workspace,
    pike_profile_begin,
    pike_profile_end,
    pike_set_wait_limit_ns,
    pike_status_string,
)
