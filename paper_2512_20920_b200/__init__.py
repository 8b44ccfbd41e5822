"""B200 (sm_100a) library for the MoE coupling branch of a RevFFN block:
forward Y2 = X2 + MLP(Norm(Y1)), its inverse, and its backward by
recomputation.  All arithmetic runs in the CUDA library behind the C ABI in
include/revffn_moe.h; this package only marshals arguments."""
from .binding import (revffn_moe_step_host, revffn_prof_enable, revffn_prof_launches, revffn_prof_collect,
                      Block, Desc, Grads, Weights, lib, revffn_moe_backward, revffn_moe_forward,
                      revffn_moe_inverse, revffn_moe_status, revffn_moe_workspace_size, revffn_strerror,
                      RevffnError, BF16, F32, NORM_RMS, NORM_NONE, FLAG_FORCE_SIMT)

__all__ = ["revffn_moe_step_host", "revffn_prof_enable", "revffn_prof_launches", "revffn_prof_collect", "Block", "Desc", "Grads", "Weights", "lib", "revffn_moe_backward", "revffn_moe_forward",
           "revffn_moe_inverse", "revffn_moe_status", "revffn_moe_workspace_size", "revffn_strerror",
           "RevffnError", "BF16", "F32", "NORM_RMS", "NORM_NONE", "FLAG_FORCE_SIMT"]
