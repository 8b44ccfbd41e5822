"""Shared helpers for the GPU parity tests (argument marshalling only)."""
from __future__ import annotations

import numpy as np
import torch

from workloads import BlockConfig


def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (den if den > 0 else 1.0))


def max_block_rel_l2(a, b, axis: int = 0):
    """Largest relative L2 error over the slices along `axis` (one expert of a stacked weight gradient,
    one token row of a stream), skipping slices whose reference is all zero (those must be all zero in `a`
    too).  A per-tensor norm cannot see one wrong slice inside a large tensor; this can."""
    a = np.moveaxis(np.asarray(a, dtype=np.float64), axis, 0)
    b = np.moveaxis(np.asarray(b, dtype=np.float64), axis, 0)
    a = a.reshape(a.shape[0], -1)
    b = b.reshape(b.shape[0], -1)
    den = np.linalg.norm(b, axis=1)
    num = np.linalg.norm(a - b, axis=1)
    zero = den == 0
    assert (num[zero] == 0).all(), "non-zero values where the reference slice is exactly zero"
    return float((num[~zero] / den[~zero]).max()) if (~zero).any() else 0.0


def to_device_weights(cfg: BlockConfig, w: dict) -> dict:
    wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
    out = {}
    for name, v in w.items():
        if v is None:
            continue
        dt = torch.float32 if name in ("norm_gamma", "b_router") else wdt
        out[name] = torch.from_numpy(np.ascontiguousarray(v)).to(device="cuda", dtype=dt).contiguous()
    return out


def make_block(cfg: BlockConfig, w: dict, *, flags: int = 0, norm_none: bool = False, ld_stream=None,
               tokens=None):
    import paper_2512_20920_b200 as rv
    return rv.Block(tokens=cfg.tokens if tokens is None else tokens, d_model=cfg.d_model, n_experts=cfg.n_experts,
                    top_k=cfg.top_k, d_expert=cfg.d_expert, d_shared=cfg.d_shared,
                    weight_dtype=rv.BF16 if cfg.weight_dtype == "bf16" else rv.F32,
                    weights=to_device_weights(cfg, w), norm_kind=rv.NORM_NONE if norm_none else rv.NORM_RMS,
                    norm_eps=cfg.norm_eps, ld_stream=ld_stream, flags=flags)


def dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def grad_buffers(cfg: BlockConfig, w: dict, fill: float = float("nan")) -> dict:
    return {n: torch.full(v.shape, fill, dtype=torch.float32, device="cuda") for n, v in w.items() if v is not None}
