"""B200-native GAS layer pass for full-graph GNN inference (InferTurbo, arXiv 2307.00228).

The public calls mirror the C ABI in include/inferturbo.h.
"""
from .binding import (Graph, ItError, LayerDesc, it_graph_check, it_graph_create, it_graph_destroy, it_graph_get_split,  # noqa: F401
                      it_infer, it_kernel_launch_count, it_last_error_message, it_layer_forward, it_layer_forward_static, it_profile_begin, it_profile_end, it_split_hubs, it_status_string,
                      it_workspace_bytes, lib)
