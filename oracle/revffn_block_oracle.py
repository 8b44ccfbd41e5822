"""CPU oracle for a whole RevFFN block and a stack of them.  TEST INFRASTRUCTURE.

Plain numpy, fp64.  It composes the two branch oracles exactly as Sec. 3.1 writes the block
and adds nothing of its own but the order of the steps:

  forward   Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2))          (Eq. 1)
            Y2 = X2 + MLP(Norm(Y1))                                (Eq. 2)
  inverse   X2 = Y2 - MLP(Norm(Y1))                                (Sec. 3.1, first line of the inverse pass)
            X1 = fixed point of X1 = Y1 - Attn(Norm(X1), Norm(X2), Norm(X2)), n_iter iterations from X1 = Y1
  backward  reversible back-propagation (Sec. 2): rebuild (X1, X2) from (Y1, Y2), then push
            (dY1, dY2) through Eq. 2 and Eq. 1 in reverse order:
              dY1' = dY1 + J_mlp^T dY2,        dX2' = dY2
              dX1  = dY1' + J_attn,1^T dY1',   dX2  = dX2' + J_attn,2^T dY1'
            With `exact_inputs` the gradients are taken at the true inputs instead of the reconstructed
            ones (what a caching implementation computes); the two differ by the reconstruction error.
  stack     layer l+1 reads layer l's [Y1, Y2] as its [X1, X2] (Sec. 3.1: the halves are concatenated
            and passed to the next layer).

Imported only by the tests, the smoke check and the benchmark's CPU-baseline leg.
Pins (tests/test_oracle_block_pins.py): central differences through the whole block, exact
invertibility to 1e-10 in fp64 once the fixed point has converged, and the stack's backward against
central differences of the stack's forward.
"""
from __future__ import annotations

import numpy as np

from . import revffn_attn_oracle as attn
from . import revffn_oracle as moe

F64 = np.float64


def _akw(cfg):
    return dict(S=cfg["seq_len"], n_heads=cfg["n_heads"], n_kv_heads=cfg["n_kv_heads"], eps=cfg.get("eps", 1e-6),
                theta=cfg.get("theta", 1e6))


def forward(pa, pm, X1, X2, cfg, route_override=None):
    """Eq. 1 then Eq. 2.  cfg: seq_len, n_heads, n_kv_heads, top_k (+ eps, theta).  Returns (Y1, Y2, info)."""
    Y1 = attn.forward(pa, X1, X2, **_akw(cfg))
    Y2, info = moe.forward(pm, Y1, X2, cfg["top_k"], cfg.get("eps", 1e-6), route_override=route_override)
    return Y1, Y2, info


def inverse(pa, pm, Y1, Y2, cfg, n_iter: int = 1, route_override=None):
    """Inverse pass of Sec. 3.1.  Returns (X1, X2)."""
    X2, _ = moe.inverse(pm, Y1, Y2, cfg["top_k"], cfg.get("eps", 1e-6), route_override=route_override)
    X1 = attn.inverse(pa, Y1, X2, n_iter=n_iter, **_akw(cfg))
    return X1, X2


def backward(pa, pm, Y1, Y2, dY1, dY2, cfg, n_iter: int = 1, route_override=None, exact_inputs=None):
    """Returns (X1, X2, dX1, dX2, grads_attn, grads_moe)."""
    eps, k = cfg.get("eps", 1e-6), cfg["top_k"]
    if exact_inputs is None:
        X1, X2 = inverse(pa, pm, Y1, Y2, cfg, n_iter, route_override)
    else:
        X1, X2 = (np.asarray(a, dtype=F64) for a in exact_inputs)
    gm = moe.backward(pm, Y1, dY2, k, eps, route_override=route_override)
    dY1t = np.asarray(dY1, dtype=F64) + gm["dy1"]
    dX1, dX2a, ga = attn.backward(pa, X1, X2, dY1t, **_akw(cfg))
    return X1, X2, dX1, np.asarray(dY2, dtype=F64) + dX2a, ga, gm


def stack_forward(blocks, X1, X2, cfg, route_overrides=None):
    """blocks: list of (attention weights, MoE weights).  Returns (Y1, Y2, infos)."""
    A, B = np.array(X1, dtype=F64), np.array(X2, dtype=F64)
    infos = []
    for l, (pa, pm) in enumerate(blocks):
        A, B, info = forward(pa, pm, A, B, cfg, None if route_overrides is None else route_overrides[l])
        infos.append(info)
    return A, B, infos


def stack_backward(blocks, Y1, Y2, dY1, dY2, cfg, n_iter: int = 1, route_overrides=None):
    """Reversible back-propagation through the stack.  Returns (X1, X2, dX1, dX2, grads) with
    grads[l] = (attention gradients, MoE gradients) of layer l."""
    A, B = np.array(Y1, dtype=F64), np.array(Y2, dtype=F64)
    gA, gB = np.array(dY1, dtype=F64), np.array(dY2, dtype=F64)
    grads = [None] * len(blocks)
    for l in reversed(range(len(blocks))):
        pa, pm = blocks[l]
        A, B, gA, gB, ga, gm = backward(pa, pm, A, B, gA, gB, cfg, n_iter,
                                        None if route_overrides is None else route_overrides[l])
        grads[l] = (ga, gm)
    return A, B, gA, gB, grads
