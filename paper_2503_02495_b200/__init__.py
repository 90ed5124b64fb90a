"""Union-of-Experts routed hot path for B200: Python binding of the C-ABI library libuoe.so.

Importing the package loads the shared library and fails if it has not been built
(`python paper_2503_02495_b200/build.py`).  There is no CPU or PyTorch fallback.
"""
from .binding import (  # noqa: F401
    LIB_PATH, Problem, Routing, UoeError, alloc_routing, alloc_saved_h, alloc_workspace, status_string,
    uoe_launch_count, uoe_tensor_map_encodings, uoe_profile_enable, uoe_profile_records, uoe_max_routed_rows, uoe_mlp_backward, uoe_mlp_forward, uoe_read_device_status, uoe_route, uoe_route_balance, uoe_route_balance_backward, uoe_route_static, UOE_OP_BALANCE_BWD, UOE_ROUTE_STATIC_SCRATCH_BYTES,
    uoe_smha_forward, uoe_smha_backward, uoe_workspace_bytes, UOE_OP_ROUTE, UOE_OP_MLP_FWD, UOE_OP_MLP_BWD, UOE_OP_SMHA_FWD,
    UOE_OP_SMHA_BWD,
    UOE_ROW_ALIGN, alloc_block_workspace, uoe_block_forward, uoe_block_workspace_bytes,
)
