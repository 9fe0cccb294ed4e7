"""B200-native WERSA attention operator (arXiv 2507.08637): ctypes binding of the CUDA library."""
from .binding import (WERSA_BF16, WERSA_F32, WERSA_FLAG_FORWARD_ONLY, WERSA_FLAG_SIMT_ONLY, LIB_PATH,
                      WersaContext, WersaError, make_config, wersa_backward, wersa_config, wersa_create,
                      wersa_destroy, wersa_forward, wersa_forward_host, wersa_gate_static, wersa_status_string,
                      wersa_workspace_bytes)

__all__ = ["WERSA_BF16", "WERSA_F32", "WERSA_FLAG_FORWARD_ONLY", "WERSA_FLAG_SIMT_ONLY", "LIB_PATH",
           "WersaContext", "WersaError", "make_config", "wersa_backward", "wersa_config", "wersa_create",
           "wersa_destroy", "wersa_forward", "wersa_forward_host", "wersa_gate_static", "wersa_status_string", "wersa_workspace_bytes"]
