"""B200-native (sm_100a) library for the decode-time W2A4 hot path of RCP (arXiv 2502.15779):
weight-code packing, fused Hadamard + int4 activation quantization, and the LUT GEMV.

The compute lives in ``librcp_w2a4.so`` (hand-written CUDA behind the C ABI of include/rcp.h);
this package only marshals arguments. Importing it needs neither a GPU nor the built library;
calling any entry point without the library raises.
"""
from .binding import (RcpError, lib, make_workspace, rcp_gemv_w2a4, rcp_gemv_workspace_bytes,  # noqa: F401
                      rcp_gemv_w2a4_grouped, rcp_gemv_w2a4_static, rcp_gemv_w2a16, rcp_ldp_export, rcp_nf3_export, rcp_linear_w2a4, rcp_linear_w2a4_host, rcp_linear_w2a4_launches, rcp_pack_weights, rcp_quantize_act,
                      rcp_pack_weights3, rcp_gemv_w3a4)
