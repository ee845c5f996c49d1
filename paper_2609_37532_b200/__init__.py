"""B200-native DScale verify path: thin Python binding over libdscale.so.

Every step of the path runs in the CUDA library; this package only marshals
torch tensors (device memory, streams) into the C ABI declared in
include/dscale.h.  There is no CPU fallback: importing the binding without the
built library raises.
"""
from .build import build as _build

_build()          # no-op when libdscale.so is newer than its sources; raises if nvcc fails

from .binding import (  # noqa: E402
    DScaleError, HostStep, VerifyGraphPool, VerifyWorkspace, accept, accept_sampling, accept_static, alloc_verify, lib, lm_head_accept, predict_scores, verify_attn,
                      verify_attn_padded, verify_attn_simt, WS_FIELDS)

__all__ = ["DScaleError", "HostStep", "VerifyGraphPool", "VerifyWorkspace", "accept", "accept_sampling", "accept_static", "alloc_verify", "lib", "lm_head_accept", "predict_scores", "verify_attn",
           "verify_attn_padded", "verify_attn_simt", "WS_FIELDS"]
