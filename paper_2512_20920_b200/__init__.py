"""B200 (sm_100a) library for the coupling branches of a RevFFN block: the MoE branch
Y2 = X2 + MLP(Norm(Y1)) and the attention branch Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2)),
each with its inverse and its backward by recomputation.  All arithmetic runs in the CUDA
library behind the C ABI in include/revffn_moe.h and include/revffn_attn.h; this package only
marshals arguments.

Names are resolved from `binding` on first use, so that `build` can be imported
before the shared library exists.  There is no fallback: using anything here
without the built library raises ImportError."""
import importlib

__all__ = ["Block", "Stack", "revffn_moe_saved_size", "revffn_moe_stack_cache_stride",
           "revffn_moe_stack_forward", "revffn_moe_stack_backward", "Desc", "Grads", "Weights", "lib", "revffn_moe_backward", "revffn_moe_forward",
           "revffn_moe_inverse", "revffn_moe_status", "revffn_moe_workspace_size", "revffn_strerror",
           "revffn_moe_step_host", "revffn_moe_route_noalloc", "revffn_prof_enable", "revffn_prof_launches",
           "revffn_prof_collect", "RevffnError", "BF16", "F32", "NORM_RMS", "NORM_NONE", "FLAG_FORCE_SIMT",
           "FLAG_SAVE_ACTIVATIONS", "FLAG_REUSE_ACTIVATIONS", "FLAG_GATE_SOFTMAX_ALL", "FLAG_ROUTING_RECORD",
           "FLAG_KEEP_STATUS", "FLAG_FP8_EXPERTS", "FLAG_STEP_PIPELINED", "FLAG_SINGLE_STREAM", "FLAG_DEBUG_CHECKS", "FLAG_ROUTER_FOLDED", "ERR_DEVICE_WAIT", "ERR_UNSUPPORTED",
           "ERR_NOALLOC_LIMIT", "ERR_INDEX", "Sgd", "make_sgd", "upd_mask", "UPD_NAMES", "UPD_ALL", "stage_update_mask",
           "revffn_moe_backward_sgd", "revffn_moe_backward_adam", "revffn_moe_stack_backward_adam", "Adam", "make_adam", "revffn_moe_stack_backward_sgd", "ERR_CANARY", "ERR_NONFINITE", "revffn_dbg_check_guards", "ws_lookup",
           "revffn_moe_routing_record_bytes", "AttnBranch", "AttnDesc", "AttnWeights", "AttnGrads",
           "revffn_attn_workspace_size", "revffn_attn_forward", "revffn_attn_inverse", "revffn_attn_backward",
           "revffn_attn_status", "BlockDesc", "RevStack", "revffn_block_workspace_size", "revffn_block_forward",
           "revffn_block_inverse", "revffn_block_backward", "revffn_block_stack_forward", "revffn_block_stack_backward",
           "revffn_block_status", "trainable_names"]


def __getattr__(name):
    if name in __all__:
        return getattr(importlib.import_module(".binding", __name__), name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
