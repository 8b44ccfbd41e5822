"""ctypes binding of librevffn_moe.so: the same entry points as
include/revffn_moe.h, include/revffn_attn.h and include/revffn_block.h, taking torch tensors for device memory and the current
torch CUDA stream.  Argument marshalling only; no arithmetic happens here, and
there is no fallback: a missing library is an ImportError."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librevffn_moe.so")

F32, BF16 = 0, 1
NORM_RMS, NORM_NONE = 0, 1
FLAG_FORCE_SIMT = 1
FLAG_SAVE_ACTIVATIONS = 2
FLAG_REUSE_ACTIVATIONS = 4
FLAG_GATE_SOFTMAX_ALL = 8
FLAG_ROUTING_RECORD = 16
FLAG_KEEP_STATUS = 32
FLAG_DEBUG_CHECKS = 64
FLAG_ROUTER_FOLDED = 128
FLAG_FP8_EXPERTS = 256
FLAG_STEP_PIPELINED = 512
FLAG_SINGLE_STREAM = 1024

ERR_DEVICE_WAIT, ERR_UNSUPPORTED, ERR_NOALLOC_LIMIT, ERR_INDEX, ERR_CANARY, ERR_NONFINITE = -7, -8, -9, -10, -11, -12

WEIGHT_NAMES = ("norm_gamma", "w_up", "w_down", "w_router", "b_router", "w_gate", "w_upx", "w_downx",
                "ws_gate", "ws_up", "ws_down", "ws_sgate")
_F32_ALWAYS = ("norm_gamma", "b_router")


class RevffnError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {revffn_strerror(code)} ({code})")
        self.code = code


class Desc(C.Structure):
    _fields_ = [("tokens", C.c_int32), ("d_model", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32),
                ("d_expert", C.c_int32), ("d_shared", C.c_int32), ("weight_dtype", C.c_int32),
                ("norm_kind", C.c_int32), ("norm_eps", C.c_float), ("ld_stream", C.c_int64), ("flags", C.c_uint32)]


FP8_NAMES = ("q_gate", "q_upx", "q_downx", "s_gate", "s_upx", "s_downx")      # e4m3 codes and fp32 row scales of the experts


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES + FP8_NAMES]


class Grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES] + [("accumulate", C.c_int32)]


UPD_NAMES = ("w_up", "w_down", "w_gate", "w_upx", "w_downx", "ws_gate", "ws_up", "ws_down")     # bit i of the mask
UPD_ALL = 255


class Sgd(C.Structure):
    """revffn_moe_sgd: learning rate, mask of the matrices updated in place, optional fp32 master copies."""
    _fields_ = [("lr", C.c_float), ("mask", C.c_uint32)] + [("m_" + n, C.c_void_p) for n in UPD_NAMES]


def upd_mask(names) -> int:
    """REVFFN_UPD_* mask of the named matrices."""
    return sum(1 << UPD_NAMES.index(n) for n in names)


def make_sgd(lr: float, names, masters: Optional[Dict[str, torch.Tensor]] = None) -> Sgd:
    masters = masters or {}
    for n, t in masters.items():
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
            raise ValueError(f"master copy {n}: need a contiguous fp32 CUDA tensor")
    return Sgd(lr=lr, mask=upd_mask(names), **{"m_" + n: _ptr(masters.get(n)) for n in UPD_NAMES})


class Adam(C.Structure):
    """revffn_moe_adam: the rule's constants, the caller's step counter, mask, moment buffers and optional fp32
    master copies (arrays indexed by the position of the matrix in UPD_NAMES)."""
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int32), ("mask", C.c_uint32), ("mom", C.c_void_p * 8),
                ("var", C.c_void_p * 8), ("master", C.c_void_p * 8)]


def make_adam(lr: float, step: int, names, mom: Dict[str, torch.Tensor], var: Dict[str, torch.Tensor],
              masters: Optional[Dict[str, torch.Tensor]] = None, beta1: float = 0.9, beta2: float = 0.999,
              eps: float = 1e-8, weight_decay: float = 0.0) -> Adam:
    masters = masters or {}
    for d in (mom, var, masters):
        for n, t in d.items():
            if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"{n}: need a contiguous fp32 CUDA tensor")
    a = Adam(lr=lr, beta1=beta1, beta2=beta2, eps=eps, weight_decay=weight_decay, step=step, mask=upd_mask(names))
    for i, n in enumerate(UPD_NAMES):
        a.mom[i], a.var[i], a.master[i] = _ptr(mom.get(n)), _ptr(var.get(n)), _ptr(masters.get(n))
    return a


ATTN_WEIGHT_NAMES = ("norm_gamma", "w_up", "w_down", "w_q", "w_k", "w_v", "w_o", "b_q", "b_k", "b_v")
_ATTN_F32_ALWAYS = ("norm_gamma", "b_q", "b_k", "b_v")


class AttnDesc(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq_len", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("weight_dtype", C.c_int32), ("norm_eps", C.c_float),
                ("rope_theta", C.c_float), ("ld_stream", C.c_int64), ("flags", C.c_uint32)]


class AttnWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ATTN_WEIGHT_NAMES]


class AttnGrads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ATTN_WEIGHT_NAMES] + [("accumulate", C.c_int32)]


class BlockDesc(C.Structure):
    _fields_ = [("attn", AttnDesc), ("moe", Desc), ("inverse_iters", C.c_int32)]


class DbgGemmArgs(C.Structure):
    _fields_ = [("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32), ("a_mn_major", C.c_int32),
                ("b_mn_major", C.c_int32), ("concat", C.c_int32), ("epilogue", C.c_int32), ("out_f32", C.c_int32),
                ("accumulate", C.c_int32), ("use_simt", C.c_int32), ("A", C.c_void_p), ("B0", C.c_void_p),
                ("B1", C.c_void_p), ("lda", C.c_int64), ("ldb", C.c_int64), ("C", C.c_void_p), ("C1", C.c_void_p),
                ("ldc", C.c_int64), ("ldc1", C.c_int64), ("rowscale", C.c_void_p), ("resid", C.c_void_p),
                ("ld_resid", C.c_int64), ("resid_sign", C.c_float), ("ab", C.c_void_p), ("ld_ab", C.c_int64),
                ("dg_part", C.c_void_p), ("dg_ld", C.c_int32), ("group_mode", C.c_int32), ("n_groups", C.c_int32),
                ("group_off", C.c_void_p), ("tile_group", C.c_void_p), ("rows_total", C.c_void_p),
                ("b_group_stride", C.c_int64), ("c_group_stride", C.c_int64), ("a_col0", C.c_int32),
                ("b_col0", C.c_int32), ("tok_chunks", C.c_void_p), ("no_pair", C.c_int32),
                ("wait_cycles", C.c_int64), ("starve_operands", C.c_int32), ("split_loads", C.c_int32), ("mn_boxes", C.c_int32)]


def _load() -> C.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2512_20920_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    vp, sz = C.c_void_p, C.c_size_t
    lib.revffn_moe_workspace_size.argtypes = [C.POINTER(Desc), C.POINTER(sz), C.POINTER(sz)]
    lib.revffn_moe_forward.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, vp, vp, sz, vp]
    lib.revffn_moe_inverse.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, vp, vp, sz, vp]
    lib.revffn_moe_backward.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, C.POINTER(Grads), vp, vp,
                                        sz, vp]
    lib.revffn_moe_backward_sgd.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, C.POINTER(Grads), C.POINTER(Sgd),
                                            vp, vp, sz, vp]
    lib.revffn_moe_backward_sgd.restype = C.c_int
    lib.revffn_moe_backward_adam.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, C.POINTER(Grads), C.POINTER(Adam),
                                             vp, vp, sz, vp]
    lib.revffn_moe_backward_adam.restype = C.c_int
    lib.revffn_moe_stack_backward_sgd.argtypes = [C.POINTER(Desc), C.POINTER(Weights), C.c_int32, vp, vp, vp, vp,
                                                  C.POINTER(Grads), C.POINTER(Sgd), vp, vp, sz, vp, sz, vp]
    lib.revffn_moe_stack_backward_sgd.restype = C.c_int
    lib.revffn_moe_stack_backward_adam.argtypes = [C.POINTER(Desc), C.POINTER(Weights), C.c_int32, vp, vp, vp, vp,
                                                   C.POINTER(Grads), C.POINTER(Adam), vp, vp, sz, vp, sz, vp]
    lib.revffn_moe_stack_backward_adam.restype = C.c_int
    lib.revffn_moe_quantize_experts.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp]
    lib.revffn_moe_quantize_experts.restype = C.c_int
    lib.revffn_moe_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    lib.revffn_strerror.argtypes = [C.c_int]
    lib.revffn_strerror.restype = C.c_char_p
    lib.revffn_moe_ws_lookup.argtypes = [C.POINTER(Desc), C.c_char_p, C.POINTER(sz), C.POINTER(sz)]
    lib.revffn_dbg_gemm.argtypes = [C.POINTER(DbgGemmArgs), vp, vp]
    lib.revffn_dbg_check_guards.argtypes = [C.POINTER(Desc), vp, sz, vp]
    lib.revffn_dbg_check_guards.restype = C.c_int
    lib.revffn_moe_step_host.argtypes = [C.POINTER(Desc), C.POINTER(Weights), C.POINTER(Grads), vp, vp, vp, vp, vp, vp,
                                         vp, sz, vp, sz, vp, vp]
    lib.revffn_moe_saved_size.argtypes = [C.POINTER(Desc), C.POINTER(sz)]
    lib.revffn_moe_routing_record_bytes.argtypes = [C.POINTER(Desc), C.POINTER(sz)]
    lib.revffn_moe_routing_record_bytes.restype = C.c_int
    lib.revffn_moe_stack_cache_stride.argtypes = [C.POINTER(Desc), C.POINTER(sz)]
    lib.revffn_moe_stack_forward.argtypes = [C.POINTER(Desc), C.POINTER(Weights), C.c_int32, vp, vp, vp, vp, sz, vp, sz, vp]
    lib.revffn_moe_stack_backward.argtypes = [C.POINTER(Desc), C.POINTER(Weights), C.c_int32, vp, vp, vp, vp,
                                              C.POINTER(Grads), vp, vp, sz, vp, sz, vp]
    for f in ("revffn_moe_saved_size", "revffn_moe_stack_cache_stride", "revffn_moe_stack_forward",
              "revffn_moe_stack_backward"):
        getattr(lib, f).restype = C.c_int
    lib.revffn_moe_route_noalloc.argtypes = [C.POINTER(Desc), C.POINTER(Weights), vp, vp, vp, vp, vp]
    lib.revffn_moe_route_noalloc.restype = C.c_int
    lib.revffn_attn_workspace_size.argtypes = [C.POINTER(AttnDesc), C.POINTER(sz), C.POINTER(sz)]
    lib.revffn_attn_forward.argtypes = [C.POINTER(AttnDesc), C.POINTER(AttnWeights), vp, vp, vp, vp, sz, vp]
    lib.revffn_attn_inverse.argtypes = [C.POINTER(AttnDesc), C.POINTER(AttnWeights), vp, vp, vp, C.c_int32, vp, sz, vp]
    lib.revffn_attn_backward.argtypes = [C.POINTER(AttnDesc), C.POINTER(AttnWeights), vp, vp, vp, vp, vp,
                                         C.POINTER(AttnGrads), vp, sz, vp]
    lib.revffn_attn_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    for f in ("revffn_attn_workspace_size", "revffn_attn_forward", "revffn_attn_inverse", "revffn_attn_backward",
              "revffn_attn_status"):
        getattr(lib, f).restype = C.c_int
    bd, aw, mw, ag, mg = (C.POINTER(t) for t in (BlockDesc, AttnWeights, Weights, AttnGrads, Grads))
    lib.revffn_block_workspace_size.argtypes = [bd, C.POINTER(sz), C.POINTER(sz)]
    lib.revffn_block_forward.argtypes = [bd, aw, mw, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.revffn_block_inverse.argtypes = [bd, aw, mw, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.revffn_block_backward.argtypes = [bd, aw, mw, vp, vp, vp, vp, ag, mg, vp, vp, sz, vp]
    lib.revffn_block_stack_forward.argtypes = [bd, aw, mw, C.c_int32, vp, vp, vp, vp, sz, vp]
    lib.revffn_block_stack_backward.argtypes = [bd, aw, mw, C.c_int32, vp, vp, vp, vp, ag, mg, vp, vp, sz, vp]
    lib.revffn_block_status.argtypes = [vp, vp, C.POINTER(C.c_int32)]
    for f in ("revffn_block_workspace_size", "revffn_block_forward", "revffn_block_inverse", "revffn_block_backward",
              "revffn_block_stack_forward", "revffn_block_stack_backward", "revffn_block_status"):
        getattr(lib, f).restype = C.c_int
    lib.revffn_prof_enable.argtypes = [C.c_int]
    lib.revffn_prof_launches.argtypes = []
    lib.revffn_prof_launches.restype = C.c_longlong
    lib.revffn_prof_num_slots.argtypes = []
    lib.revffn_prof_slot_name.argtypes = [C.c_int]
    lib.revffn_prof_slot_name.restype = C.c_char_p
    lib.revffn_prof_collect.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_int32), C.c_int]
    for f in ("revffn_moe_step_host", "revffn_prof_enable", "revffn_prof_num_slots", "revffn_prof_collect"):
        getattr(lib, f).restype = C.c_int
    for f in ("revffn_moe_workspace_size", "revffn_moe_forward", "revffn_moe_inverse", "revffn_moe_backward",
              "revffn_moe_status", "revffn_moe_ws_lookup", "revffn_dbg_gemm"):
        getattr(lib, f).restype = C.c_int
    return lib


lib = _load()


def revffn_strerror(code: int) -> str:
    return lib.revffn_strerror(int(code)).decode()


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str) -> None:
    if code != 0:
        raise RevffnError(code, where)


def revffn_moe_workspace_size(desc: Desc):
    f, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib.revffn_moe_workspace_size(C.byref(desc), C.byref(f), C.byref(b)), "revffn_moe_workspace_size")
    return f.value, b.value


def revffn_moe_forward(desc: Desc, w: Weights, y1, x2, y2, topk_idx_out, ws, stream: Optional[int] = None):
    _check(lib.revffn_moe_forward(C.byref(desc), C.byref(w), _ptr(y1), _ptr(x2), _ptr(y2), _ptr(topk_idx_out),
                                  _ptr(ws), ws.numel() * ws.element_size(), stream if stream is not None else _stream()),
           "revffn_moe_forward")


def revffn_moe_inverse(desc: Desc, w: Weights, y1, y2, x2, topk_idx_in, ws, stream: Optional[int] = None):
    _check(lib.revffn_moe_inverse(C.byref(desc), C.byref(w), _ptr(y1), _ptr(y2), _ptr(x2), _ptr(topk_idx_in),
                                  _ptr(ws), ws.numel() * ws.element_size(), stream if stream is not None else _stream()),
           "revffn_moe_inverse")


def revffn_moe_backward(desc: Desc, w: Weights, y1, dy2, dy1_inout, grads: Grads, topk_idx_in, ws,
                        stream: Optional[int] = None):
    _check(lib.revffn_moe_backward(C.byref(desc), C.byref(w), _ptr(y1), _ptr(dy2), _ptr(dy1_inout), C.byref(grads),
                                   _ptr(topk_idx_in), _ptr(ws), ws.numel() * ws.element_size(),
                                   stream if stream is not None else _stream()),
           "revffn_moe_backward")


def revffn_moe_backward_sgd(desc: Desc, w: Weights, y1, dy2, dy1_inout, grads: Grads, sgd: Sgd, topk_idx_in, ws,
                            stream: Optional[int] = None):
    _check(lib.revffn_moe_backward_sgd(C.byref(desc), C.byref(w), _ptr(y1), _ptr(dy2), _ptr(dy1_inout), C.byref(grads),
                                       C.byref(sgd), _ptr(topk_idx_in), _ptr(ws), ws.numel() * ws.element_size(),
                                       stream if stream is not None else _stream()),
           "revffn_moe_backward_sgd")


def revffn_moe_backward_adam(desc: Desc, w: Weights, y1, dy2, dy1_inout, grads: Grads, adam: Adam, topk_idx_in, ws,
                             stream: Optional[int] = None):
    _check(lib.revffn_moe_backward_adam(C.byref(desc), C.byref(w), _ptr(y1), _ptr(dy2), _ptr(dy1_inout), C.byref(grads),
                                        C.byref(adam), _ptr(topk_idx_in), _ptr(ws), ws.numel() * ws.element_size(),
                                        stream if stream is not None else _stream()),
           "revffn_moe_backward_adam")


def revffn_moe_status(ws, stream: Optional[int] = None) -> int:
    out = C.c_int32(0)
    _check(lib.revffn_moe_status(_ptr(ws), stream if stream is not None else _stream(), C.byref(out)),
           "revffn_moe_status")
    return out.value


def revffn_moe_step_host(desc: Desc, w: Weights, grads: Grads, y1_host, x2_host, dy2_host, y2_host, x2_rec_host,
                         dy1_host, staging, ws, stream: Optional[int] = None, copy_stream: Optional[int] = None,
                         pipelined: bool = False):
    """Host-resident streams (pinned CPU tensors) in and out; see the header.  copy_stream: raw handle of a
    second CUDA stream for the transfers that can run beside the passes, or None.  pipelined: the call is made
    with FLAG_STEP_PIPELINED (12 staging slots, results complete when copy_stream completes)."""
    if pipelined:
        d2 = Desc()
        C.memmove(C.byref(d2), C.byref(desc), C.sizeof(Desc))
        d2.flags |= FLAG_STEP_PIPELINED
        desc = d2
    _check(lib.revffn_moe_step_host(C.byref(desc), C.byref(w), C.byref(grads), _ptr(y1_host), _ptr(x2_host),
                                    _ptr(dy2_host), _ptr(y2_host), _ptr(x2_rec_host), _ptr(dy1_host), _ptr(staging),
                                    staging.numel() * staging.element_size(), _ptr(ws),
                                    ws.numel() * ws.element_size(), stream if stream is not None else _stream(),
                                    copy_stream),
           "revffn_moe_step_host")


def revffn_moe_route_noalloc(desc: Desc, w: Weights, y1, topk_idx_out, gates_out, sgate_out,
                             stream: Optional[int] = None):
    """Routing (expert indices, gate weights, shared gate) with the library's own fixed scratch: for callers
    that cannot allocate a workspace.  Calls on one device must not overlap; see the header."""
    _check(lib.revffn_moe_route_noalloc(C.byref(desc), C.byref(w), _ptr(y1), _ptr(topk_idx_out), _ptr(gates_out),
                                        _ptr(sgate_out), stream if stream is not None else _stream()),
           "revffn_moe_route_noalloc")


def revffn_moe_saved_size(desc: Desc) -> int:
    n = C.c_size_t(0)
    _check(lib.revffn_moe_saved_size(C.byref(desc), C.byref(n)), "revffn_moe_saved_size")
    return n.value


def revffn_moe_routing_record_bytes(desc: Desc) -> int:
    n = C.c_size_t(0)
    _check(lib.revffn_moe_routing_record_bytes(C.byref(desc), C.byref(n)), "revffn_moe_routing_record_bytes")
    return n.value


def revffn_moe_stack_cache_stride(desc: Desc) -> int:
    n = C.c_size_t(0)
    _check(lib.revffn_moe_stack_cache_stride(C.byref(desc), C.byref(n)), "revffn_moe_stack_cache_stride")
    return n.value


def _nbytes(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def revffn_moe_stack_forward(desc: Desc, weights, n_blocks: int, stream_a, stream_b, topk_idx, cache, ws,
                             stream: Optional[int] = None):
    """`weights` is a ctypes array of n_blocks Weights structs."""
    _check(lib.revffn_moe_stack_forward(C.byref(desc), weights, n_blocks, _ptr(stream_a), _ptr(stream_b),
                                        _ptr(topk_idx), _ptr(cache), _nbytes(cache), _ptr(ws), _nbytes(ws),
                                        stream if stream is not None else _stream()), "revffn_moe_stack_forward")


def revffn_moe_stack_backward(desc: Desc, weights, n_blocks: int, stream_a, stream_b, grad_a, grad_b, grads,
                              topk_idx, cache, ws, stream: Optional[int] = None):
    """`weights` / `grads`: ctypes arrays of n_blocks Weights / Grads structs."""
    _check(lib.revffn_moe_stack_backward(C.byref(desc), weights, n_blocks, _ptr(stream_a), _ptr(stream_b),
                                         _ptr(grad_a), _ptr(grad_b), grads, _ptr(topk_idx), _ptr(cache),
                                         _nbytes(cache), _ptr(ws), _nbytes(ws),
                                         stream if stream is not None else _stream()), "revffn_moe_stack_backward")


def revffn_moe_stack_backward_sgd(desc: Desc, weights, n_blocks: int, stream_a, stream_b, grad_a, grad_b, grads, sgd,
                                  topk_idx, cache, ws, stream: Optional[int] = None):
    """`sgd`: ctypes array of n_blocks Sgd structs (or None)."""
    _check(lib.revffn_moe_stack_backward_sgd(C.byref(desc), weights, n_blocks, _ptr(stream_a), _ptr(stream_b),
                                             _ptr(grad_a), _ptr(grad_b), grads, sgd, _ptr(topk_idx), _ptr(cache),
                                             _nbytes(cache), _ptr(ws), _nbytes(ws),
                                             stream if stream is not None else _stream()), "revffn_moe_stack_backward_sgd")


def revffn_moe_stack_backward_adam(desc: Desc, weights, n_blocks: int, stream_a, stream_b, grad_a, grad_b, grads, adam,
                                   topk_idx, cache, ws, stream: Optional[int] = None):
    """`adam`: ctypes array of n_blocks Adam structs."""
    _check(lib.revffn_moe_stack_backward_adam(C.byref(desc), weights, n_blocks, _ptr(stream_a), _ptr(stream_b),
                                              _ptr(grad_a), _ptr(grad_b), grads, adam, _ptr(topk_idx), _ptr(cache),
                                              _nbytes(cache), _ptr(ws), _nbytes(ws),
                                              stream if stream is not None else _stream()), "revffn_moe_stack_backward_adam")


def revffn_prof_enable(on: bool) -> bool:
    return bool(lib.revffn_prof_enable(1 if on else 0))


def revffn_prof_launches() -> int:
    return int(lib.revffn_prof_launches())


def revffn_prof_collect() -> Dict[str, tuple]:
    """{slot name: (total device ms, launches)} since profiling was enabled or last collected."""
    n = lib.revffn_prof_num_slots()
    ms = (C.c_float * n)()
    cnt = (C.c_int32 * n)()
    _check(lib.revffn_prof_collect(ms, cnt, n), "revffn_prof_collect")
    return {lib.revffn_prof_slot_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i] > 0}


def revffn_dbg_check_guards(desc: Desc, ws, stream: Optional[int] = None) -> None:
    """Verify the workspace's guard zones now (desc must carry FLAG_DEBUG_CHECKS); the result is in the status word."""
    _check(lib.revffn_dbg_check_guards(C.byref(desc), _ptr(ws), ws.numel() * ws.element_size(),
                                       stream if stream is not None else _stream()), "revffn_dbg_check_guards")


def ws_lookup(desc: Desc, name: str):
    off, nbytes = C.c_size_t(0), C.c_size_t(0)
    _check(lib.revffn_moe_ws_lookup(C.byref(desc), name.encode(), C.byref(off), C.byref(nbytes)), "revffn_moe_ws_lookup")
    return off.value, nbytes.value


class Block:
    """One block's descriptor, device weights and workspace, with the three
    passes as methods.  Pure marshalling around the C entry points."""

    def __init__(self, *, tokens: int, d_model: int, n_experts: int, top_k: int, d_expert: int, d_shared: int,
                 weight_dtype: int, weights: Dict[str, torch.Tensor], norm_kind: int = NORM_RMS,
                 norm_eps: float = 1e-6, ld_stream: Optional[int] = None, flags: int = 0,
                 workspace: Optional[torch.Tensor] = None, backward: bool = True):
        self.desc = Desc(tokens, d_model, n_experts, top_k, d_expert, d_shared, weight_dtype, norm_kind, norm_eps,
                         ld_stream if ld_stream is not None else d_model // 2, flags)
        wdt = torch.bfloat16 if weight_dtype == BF16 else torch.float32
        self.weights = {}
        for name in WEIGHT_NAMES:
            t = weights.get(name)
            if t is None:
                continue
            want = torch.float32 if name in _F32_ALWAYS else wdt
            if t.dtype != want or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"weight {name}: need a contiguous CUDA tensor of {want}")
            self.weights[name] = t
        self.w = Weights(**{n: _ptr(self.weights.get(n)) for n in WEIGHT_NAMES})
        self.fwd_bytes, self.bwd_bytes = revffn_moe_workspace_size(self.desc)
        need = self.bwd_bytes if backward else self.fwd_bytes
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device="cuda")
        if workspace.numel() * workspace.element_size() < need:
            raise ValueError("workspace too small")
        self.ws = workspace

    @property
    def tokens(self) -> int:
        return self.desc.tokens

    def quantize_experts(self) -> Dict[str, torch.Tensor]:
        """Buffers for the e4m3 copies of the expert weights and their row scales, filled by
        revffn_moe_quantize_experts and entered into this block's weight struct (needed with FLAG_FP8_EXPERTS)."""
        E, I, d = self.desc.n_experts, self.desc.d_expert, self.desc.d_model
        q = {"q_gate": torch.empty(E, I, d, dtype=torch.uint8, device="cuda"),
             "q_upx": torch.empty(E, I, d, dtype=torch.uint8, device="cuda"),
             "q_downx": torch.empty(E, d, I, dtype=torch.uint8, device="cuda"),
             "s_gate": torch.empty(E, I, dtype=torch.float32, device="cuda"),
             "s_upx": torch.empty(E, I, dtype=torch.float32, device="cuda"),
             "s_downx": torch.empty(E, d, dtype=torch.float32, device="cuda")}
        for n, t in q.items():
            setattr(self.w, n, _ptr(t))
        self.fp8 = q
        _check(lib.revffn_moe_quantize_experts(C.byref(self.desc), C.byref(self.w), _stream()), "revffn_moe_quantize_experts")
        return q

    def _desc(self, extra_flags: int) -> Desc:
        if not extra_flags:
            return self.desc
        d = Desc()
        C.memmove(C.byref(d), C.byref(self.desc), C.sizeof(Desc))
        d.flags = self.desc.flags | extra_flags
        return d

    def forward(self, y1, x2, y2=None, topk_idx_out=None, save: bool = False, ws=None, flags: int = 0):
        """save=True keeps the branch's intermediates for a later backward(reuse=True); flags: more REVFFN_FLAG_* bits
        for this call (e.g. FLAG_ROUTER_FOLDED, FLAG_KEEP_STATUS)."""
        if y2 is None:
            y2 = torch.empty_like(x2)
        revffn_moe_forward(self._desc((FLAG_SAVE_ACTIVATIONS if save else 0) | flags), self.w, y1, x2, y2, topk_idx_out,
                           self.ws if ws is None else ws)
        return y2

    def inverse(self, y1, y2, x2=None, topk_idx_in=None, save: bool = False, ws=None, flags: int = 0):
        if x2 is None:
            x2 = torch.empty_like(y2)
        revffn_moe_inverse(self._desc((FLAG_SAVE_ACTIVATIONS if save else 0) | flags), self.w, y1, y2, x2, topk_idx_in,
                           self.ws if ws is None else ws)
        return x2

    def backward(self, y1, dy2, dy1_inout, grads: Optional[Dict[str, torch.Tensor]] = None, accumulate: bool = False,
                 topk_idx_in=None, reuse: bool = False, ws=None, flags: int = 0, sgd: Optional[Sgd] = None):
        """reuse=True: the workspace still holds what forward/inverse(save=True) left for this y1.
        sgd: a Sgd struct (make_sgd) or an Adam struct (make_adam) -- the matrices in its mask are updated in place
        instead of having their gradients written (revffn_moe_backward_sgd / revffn_moe_backward_adam)."""
        grads = grads or {}
        for n, t in grads.items():
            if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"gradient {n}: need a contiguous fp32 CUDA tensor")
        g = Grads(**{n: _ptr(grads.get(n)) for n in WEIGHT_NAMES}, accumulate=1 if accumulate else 0)
        d = self._desc((FLAG_REUSE_ACTIVATIONS if reuse else 0) | flags)
        if isinstance(sgd, Adam):
            revffn_moe_backward_adam(d, self.w, y1, dy2, dy1_inout, g, sgd, topk_idx_in, self.ws if ws is None else ws)
        elif sgd is not None:
            revffn_moe_backward_sgd(d, self.w, y1, dy2, dy1_inout, g, sgd, topk_idx_in, self.ws if ws is None else ws)
        else:
            revffn_moe_backward(d, self.w, y1, dy2, dy1_inout, g, topk_idx_in, self.ws if ws is None else ws)
        return dy1_inout

    def grads_struct(self, grads: Optional[Dict[str, torch.Tensor]] = None, accumulate: bool = False) -> Grads:
        grads = grads or {}
        return Grads(**{n: _ptr(grads.get(n)) for n in WEIGHT_NAMES}, accumulate=1 if accumulate else 0)

    def status(self) -> int:
        return revffn_moe_status(self.ws)

    def buffer(self, name: str, dtype: torch.dtype) -> torch.Tensor:
        """A named intermediate inside the workspace (tests only)."""
        off, nbytes = ws_lookup(self.desc, name)
        return self.ws[off:off + nbytes].view(dtype)


def _nb(t) -> int:
    return t.numel() * t.element_size()


def revffn_attn_workspace_size(desc: AttnDesc):
    f, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib.revffn_attn_workspace_size(C.byref(desc), C.byref(f), C.byref(b)), "revffn_attn_workspace_size")
    return f.value, b.value


def revffn_attn_forward(desc: AttnDesc, w: AttnWeights, x1, x2, y1, ws, stream: Optional[int] = None):
    _check(lib.revffn_attn_forward(C.byref(desc), C.byref(w), _ptr(x1), _ptr(x2), _ptr(y1), _ptr(ws), _nb(ws),
                                   stream if stream is not None else _stream()), "revffn_attn_forward")


def revffn_attn_inverse(desc: AttnDesc, w: AttnWeights, y1, x2, x1, n_iter: int, ws, stream: Optional[int] = None):
    _check(lib.revffn_attn_inverse(C.byref(desc), C.byref(w), _ptr(y1), _ptr(x2), _ptr(x1), int(n_iter), _ptr(ws),
                                   _nb(ws), stream if stream is not None else _stream()), "revffn_attn_inverse")


def revffn_attn_backward(desc: AttnDesc, w: AttnWeights, x1, x2, dy1, dx1, dx2_inout, grads: AttnGrads, ws,
                         stream: Optional[int] = None):
    _check(lib.revffn_attn_backward(C.byref(desc), C.byref(w), _ptr(x1), _ptr(x2), _ptr(dy1), _ptr(dx1),
                                    _ptr(dx2_inout), C.byref(grads), _ptr(ws), _nb(ws),
                                    stream if stream is not None else _stream()), "revffn_attn_backward")


def revffn_attn_status(ws, stream: Optional[int] = None) -> int:
    out = C.c_int32(0)
    _check(lib.revffn_attn_status(_ptr(ws), stream if stream is not None else _stream(), C.byref(out)),
           "revffn_attn_status")
    return out.value


class AttnBranch:
    """Descriptor, device weights and workspace of one attention coupling branch, with the three
    passes as methods.  Pure marshalling around the C entry points."""

    def __init__(self, *, batch: int, seq_len: int, d_model: int, n_heads: int, n_kv_heads: int, weight_dtype: int,
                 weights: Dict[str, torch.Tensor], norm_eps: float = 1e-6, rope_theta: float = 1e6,
                 ld_stream: Optional[int] = None, flags: int = 0, backward: bool = True):
        self.desc = AttnDesc(batch, seq_len, d_model, n_heads, n_kv_heads, weight_dtype, norm_eps, rope_theta,
                             ld_stream if ld_stream is not None else d_model // 2, flags)
        wdt = torch.bfloat16 if weight_dtype == BF16 else torch.float32
        self.weights = {}
        for name in ATTN_WEIGHT_NAMES:
            t = weights.get(name)
            if t is None:
                continue
            want = torch.float32 if name in _ATTN_F32_ALWAYS else wdt
            if t.dtype != want or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"weight {name}: need a contiguous CUDA tensor of {want}")
            self.weights[name] = t
        self.w = AttnWeights(**{n: _ptr(self.weights.get(n)) for n in ATTN_WEIGHT_NAMES})
        self.fwd_bytes, self.bwd_bytes = revffn_attn_workspace_size(self.desc)
        self.ws = torch.empty(self.bwd_bytes if backward else self.fwd_bytes, dtype=torch.uint8, device="cuda")

    def forward(self, x1, x2, y1=None):
        if y1 is None:
            y1 = torch.empty_like(x1)
        revffn_attn_forward(self.desc, self.w, x1, x2, y1, self.ws)
        return y1

    def inverse(self, y1, x2, x1=None, n_iter: int = 1):
        if x1 is None:
            x1 = torch.empty_like(y1)
        revffn_attn_inverse(self.desc, self.w, y1, x2, x1, n_iter, self.ws)
        return x1

    def backward(self, x1, x2, dy1, dx2_inout, dx1=None, grads: Optional[Dict[str, torch.Tensor]] = None,
                 accumulate: bool = False, reuse_kv: bool = False):
        """reuse_kv=True: the workspace still holds the key/value side that inverse(n_iter >= 1) left for this x2."""
        grads = grads or {}
        for n, t in grads.items():
            if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"gradient {n}: need a contiguous fp32 CUDA tensor")
        if dx1 is None:
            dx1 = torch.empty_like(dy1)
        g = AttnGrads(**{n: _ptr(grads.get(n)) for n in ATTN_WEIGHT_NAMES}, accumulate=1 if accumulate else 0)
        d = self.desc
        if reuse_kv:
            d = AttnDesc()
            C.memmove(C.byref(d), C.byref(self.desc), C.sizeof(AttnDesc))
            d.flags |= FLAG_REUSE_ACTIVATIONS
        revffn_attn_backward(d, self.w, x1, x2, dy1, dx1, dx2_inout, g, self.ws)
        return dx1

    def status(self) -> int:
        return revffn_attn_status(self.ws)


def _st(stream):
    return stream if stream is not None else _stream()


def revffn_block_workspace_size(desc: BlockDesc):
    f, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib.revffn_block_workspace_size(C.byref(desc), C.byref(f), C.byref(b)), "revffn_block_workspace_size")
    return f.value, b.value


def revffn_block_forward(desc, wa, wm, x1, x2, y1, y2, topk_idx_out, ws, stream=None):
    _check(lib.revffn_block_forward(C.byref(desc), C.byref(wa), C.byref(wm), _ptr(x1), _ptr(x2), _ptr(y1), _ptr(y2),
                                    _ptr(topk_idx_out), _ptr(ws), _nb(ws), _st(stream)), "revffn_block_forward")


def revffn_block_inverse(desc, wa, wm, y1, y2, x1, x2, topk_idx_in, ws, stream=None):
    _check(lib.revffn_block_inverse(C.byref(desc), C.byref(wa), C.byref(wm), _ptr(y1), _ptr(y2), _ptr(x1), _ptr(x2),
                                    _ptr(topk_idx_in), _ptr(ws), _nb(ws), _st(stream)), "revffn_block_inverse")


def revffn_block_backward(desc, wa, wm, s1, s2, g1, g2, ga, gm, topk_idx_in, ws, stream=None):
    _check(lib.revffn_block_backward(C.byref(desc), C.byref(wa), C.byref(wm), _ptr(s1), _ptr(s2), _ptr(g1), _ptr(g2),
                                     C.byref(ga), C.byref(gm), _ptr(topk_idx_in), _ptr(ws), _nb(ws), _st(stream)),
           "revffn_block_backward")


def revffn_block_stack_forward(desc, wa_array, wm_array, n_blocks, s1, s2, topk_idx, ws, stream=None):
    _check(lib.revffn_block_stack_forward(C.byref(desc), wa_array, wm_array, int(n_blocks), _ptr(s1), _ptr(s2),
                                          _ptr(topk_idx), _ptr(ws), _nb(ws), _st(stream)), "revffn_block_stack_forward")


def revffn_block_stack_backward(desc, wa_array, wm_array, n_blocks, s1, s2, g1, g2, ga_array, gm_array, topk_idx, ws,
                                stream=None):
    _check(lib.revffn_block_stack_backward(C.byref(desc), wa_array, wm_array, int(n_blocks), _ptr(s1), _ptr(s2), _ptr(g1),
                                           _ptr(g2), ga_array, gm_array, _ptr(topk_idx), _ptr(ws), _nb(ws), _st(stream)),
           "revffn_block_stack_backward")


def revffn_block_status(ws, stream=None) -> int:
    out = C.c_int32(0)
    _check(lib.revffn_block_status(_ptr(ws), _st(stream), C.byref(out)), "revffn_block_status")
    return out.value


def stage_update_mask(stage: int) -> int:
    """REVFFN_UPD_* mask of the MoE branch's matrices that a stage of the schedule trains (Sec. 3.3): stage 1 the
    projection adapters, stage 2 adapters and experts (the vectors and the frozen router are never fused)."""
    return upd_mask([n for n in trainable_names(stage)[1] if n in UPD_NAMES])


def trainable_names(stage: int):
    """Which weights receive gradients in the two stages of the paper's schedule (Sec. 3.3): stage 1 trains only
    the projection adapters of both branches, stage 2 everything except the MoE router, which stays frozen.
    Returns (attention names, MoE names); gradients of the other weights are passed as NULL and skipped."""
    if stage == 1:
        return ("w_up", "w_down"), ("w_up", "w_down")
    if stage == 2:
        return tuple(ATTN_WEIGHT_NAMES), tuple(n for n in WEIGHT_NAMES if n not in ("w_router", "b_router"))
    raise ValueError("stage must be 1 or 2")


class RevStack:
    """n_blocks whole RevFFN blocks (attention branch then MoE branch per block): descriptors, per-layer device
    weights and one workspace.  Pure marshalling around revffn_block_stack_forward / _backward; a single block is
    the case n_blocks = 1."""

    def __init__(self, *, batch: int, seq_len: int, d_model: int, n_heads: int, n_kv_heads: int, n_experts: int,
                 top_k: int, d_expert: int, d_shared: int, weight_dtype: int, attn_weights, moe_weights,
                 inverse_iters: int = 1, norm_eps: float = 1e-6, rope_theta: float = 1e6, flags: int = 0,
                 moe_flags: int = 0, backward: bool = True):
        h = d_model // 2
        self.n_blocks = len(attn_weights)
        if len(moe_weights) != self.n_blocks:
            raise ValueError("one attention and one MoE weight set per block")
        self.desc = BlockDesc(AttnDesc(batch, seq_len, d_model, n_heads, n_kv_heads, weight_dtype, norm_eps, rope_theta, h,
                                       flags),
                              Desc(batch * seq_len, d_model, n_experts, top_k, d_expert, d_shared, weight_dtype, NORM_RMS,
                                   norm_eps, h, flags | moe_flags), inverse_iters)
        self._keep = (attn_weights, moe_weights)            # the structs hold raw pointers into these tensors
        self.wa = (AttnWeights * self.n_blocks)(*[AttnWeights(**{n: _ptr(w.get(n)) for n in ATTN_WEIGHT_NAMES})
                                                  for w in attn_weights])
        self.wm = (Weights * self.n_blocks)(*[Weights(**{n: _ptr(w.get(n)) for n in WEIGHT_NAMES}) for w in moe_weights])
        self.fwd_bytes, self.bwd_bytes = revffn_block_workspace_size(self.desc)
        self.ws = torch.empty(self.bwd_bytes if backward else self.fwd_bytes, dtype=torch.uint8, device="cuda")

    def with_iters(self, n: int) -> BlockDesc:
        d = BlockDesc()
        C.memmove(C.byref(d), C.byref(self.desc), C.sizeof(BlockDesc))
        d.inverse_iters = n
        return d

    def grads_arrays(self, attn_grads, moe_grads, accumulate: bool = False, stage: Optional[int] = None):
        """attn_grads / moe_grads: one dict of fp32 gradient tensors per block (blocks may share tensors).
        stage: 1 or 2 keeps only the gradients that stage of the schedule trains (Sec. 3.3)."""
        acc = 1 if accumulate else 0
        keep_a, keep_m = (ATTN_WEIGHT_NAMES, WEIGHT_NAMES) if stage is None else trainable_names(stage)
        ga = (AttnGrads * self.n_blocks)(*[AttnGrads(**{n: (_ptr(g.get(n)) if n in keep_a else None)
                                                        for n in ATTN_WEIGHT_NAMES}, accumulate=acc) for g in attn_grads])
        gm = (Grads * self.n_blocks)(*[Grads(**{n: (_ptr(g.get(n)) if n in keep_m else None) for n in WEIGHT_NAMES},
                                             accumulate=acc) for g in moe_grads])
        return ga, gm

    def forward(self, s1, s2, topk_idx=None):
        revffn_block_stack_forward(self.desc, self.wa, self.wm, self.n_blocks, s1, s2, topk_idx, self.ws)

    def backward(self, s1, s2, g1, g2, ga, gm, topk_idx=None, inverse_iters: Optional[int] = None):
        d = self.desc if inverse_iters is None else self.with_iters(inverse_iters)
        revffn_block_stack_backward(d, self.wa, self.wm, self.n_blocks, s1, s2, g1, g2, ga, gm, topk_idx, self.ws)

    def inverse_block(self, l: int, y1, y2, x1, x2, topk_idx_in=None, inverse_iters: Optional[int] = None):
        d = self.desc if inverse_iters is None else self.with_iters(inverse_iters)
        revffn_block_inverse(d, self.wa[l], self.wm[l], y1, y2, x1, x2, topk_idx_in, self.ws)

    def status(self) -> int:
        return revffn_block_status(self.ws)


class Stack:
    """n_blocks coupling branches with alternating stream roles: descriptor, per-layer device
    weights, one shared workspace and, for the activation-caching variant, the per-layer cache.
    Pure marshalling around revffn_moe_stack_forward / revffn_moe_stack_backward."""

    def __init__(self, *, tokens: int, d_model: int, n_experts: int, top_k: int, d_expert: int, d_shared: int,
                 weight_dtype: int, weights, norm_kind: int = NORM_RMS, norm_eps: float = 1e-6,
                 ld_stream: Optional[int] = None, flags: int = 0, caching: bool = False):
        self.n_blocks = len(weights)
        self.desc = Desc(tokens, d_model, n_experts, top_k, d_expert, d_shared, weight_dtype, norm_kind, norm_eps,
                         ld_stream if ld_stream is not None else d_model // 2, flags)
        wdt = torch.bfloat16 if weight_dtype == BF16 else torch.float32
        self.weights = []
        for w in weights:
            kept = {}
            for name in WEIGHT_NAMES:
                t = w.get(name)
                if t is None:
                    continue
                want = torch.float32 if name in _F32_ALWAYS else wdt
                if t.dtype != want or not t.is_cuda or not t.is_contiguous():
                    raise ValueError(f"weight {name}: need a contiguous CUDA tensor of {want}")
                kept[name] = t
            self.weights.append(kept)
        self.w = (Weights * max(self.n_blocks, 1))(*[Weights(**{n: _ptr(w.get(n)) for n in WEIGHT_NAMES})
                                                     for w in self.weights])
        self.fwd_bytes, self.bwd_bytes = revffn_moe_workspace_size(self.desc)
        self.saved_bytes = revffn_moe_saved_size(self.desc)
        self.record_bytes = revffn_moe_routing_record_bytes(self.desc)
        self.cache_stride = revffn_moe_stack_cache_stride(self.desc)
        self.ws = torch.empty(self.bwd_bytes, dtype=torch.uint8, device="cuda")
        self.cache = torch.empty(self.cache_stride * self.n_blocks, dtype=torch.uint8, device="cuda") if caching else None

    def grads_array(self, grads, accumulate: bool = False):
        """ctypes array of n_blocks Grads structs from a list of {name: fp32 CUDA tensor} (one dict per layer;
        the same dict may be given for several layers)."""
        if len(grads) != self.n_blocks:
            raise ValueError("one gradient dict per layer")
        for g in grads:
            for n, t in g.items():
                if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
                    raise ValueError(f"gradient {n}: need a contiguous fp32 CUDA tensor")
        return (Grads * max(self.n_blocks, 1))(*[Grads(**{n: _ptr(g.get(n)) for n in WEIGHT_NAMES},
                                                       accumulate=1 if accumulate else 0) for g in grads])

    def forward(self, stream_a, stream_b, topk_idx=None):
        revffn_moe_stack_forward(self.desc, self.w, self.n_blocks, stream_a, stream_b, topk_idx, self.cache, self.ws)

    def backward(self, stream_a, stream_b, grad_a, grad_b, grads_array, topk_idx=None, sgd=None):
        """sgd: list of n_blocks Sgd (or Adam) structs -- one reversible sweep then is one optimiser step of the
        whole stack."""
        if sgd is not None and len(sgd) > 0 and isinstance(sgd[0], Adam):
            if len(sgd) != self.n_blocks:
                raise ValueError("one Adam struct per layer")
            arr = (Adam * max(self.n_blocks, 1))(*sgd)
            revffn_moe_stack_backward_adam(self.desc, self.w, self.n_blocks, stream_a, stream_b, grad_a, grad_b,
                                           grads_array, arr, topk_idx, self.cache, self.ws)
            return
        if sgd is not None:
            if len(sgd) != self.n_blocks:
                raise ValueError("one Sgd struct per layer")
            arr = (Sgd * max(self.n_blocks, 1))(*sgd)
            revffn_moe_stack_backward_sgd(self.desc, self.w, self.n_blocks, stream_a, stream_b, grad_a, grad_b,
                                          grads_array, arr, topk_idx, self.cache, self.ws)
            return
        revffn_moe_stack_backward(self.desc, self.w, self.n_blocks, stream_a, stream_b, grad_a, grad_b, grads_array,
                                  topk_idx, self.cache, self.ws)

    def status(self) -> int:
        """First non-zero device status word of the shared workspace and of every cache slot."""
        st = revffn_moe_status(self.ws)
        if st == 0 and self.cache is not None:
            slot = self.cache_stride - self.bwd_bytes
            for l in range(self.n_blocks):
                st = revffn_moe_status(self.cache[l * self.cache_stride + slot:])
                if st != 0:
                    break
        return st
