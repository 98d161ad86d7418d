"""B200-native low-bit and step-routed decoder linear layers (Dynamic Mixed-Precision Routing).

The product is `libdmr.so` (C ABI, see include/dmr.h); this package is its thin Python binding
plus the seeded input generators. PyTorch only supplies device memory and streams.
"""
from . import inputs  # noqa: F401
from .binding import (  # noqa: F401
    DmrError, QFormat, OUT_BF16, OUT_F32, lib, lib_path,
    dmr_quantize, dmr_dequantize, dmr_lowbit_linear, dmr_dense_linear, dmr_routed_linear,
    dmr_route_partition, dmr_stepwise_kl, dmr_lowbit_linear_host, dmr_lowbit_linear_noalloc, dmr_workspace_bytes, dmr_launch_count, dmr_describe_dispatch, dmr_router_calibrate, dmr_router_mask, dmr_router_forward, pack_router_params, RouterCfg,
    QuantizedLinear, quantize_layer, new_workspace,
)
