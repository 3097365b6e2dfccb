"""B200-native HDT hierarchical sparse attention: thin Python binding over the libhdt C ABI.

The three calls follow the C ABI (include/hdt.h): ``hdt_build_index``, ``hdt_attn_fwd``,
``hdt_attn_bwd``.  PyTorch only provides device memory and streams; every step runs in the
CUDA kernels of ``libhdt.so``.  There is no CPU or framework fallback: importing
``paper_2407_08330_b200.binding`` without the built library raises.
"""
from .binding import (HdtError, HdtIndex, hdt_attn_bwd, hdt_attn_fwd, hdt_attn_workspace_bytes,  # noqa: F401
                      hdt_build_index, hdt_index_workspace_bytes, hdt_launch_count, lib, exported_symbols, hdt_set_option,
                      hdt_device_status, hdt_attn_fwd_static, hdt_attn_fwd_static_max_bytes, hdt_hpe,
                      hdt_hpe_workspace_bytes, hdt_cross_attn_fwd, hdt_cross_attn_bwd, hdt_cross_workspace_bytes)
