"""CPU oracle for the attention coupling branch of a RevFFN block.  TEST INFRASTRUCTURE.

Plain numpy, fp64, slow on purpose: the definition of the branch written out so that a
reader can check it against the paper by eye.  It shares no code with the CUDA library
and is imported only by the tests, the smoke check and the benchmark's CPU-baseline leg;
the product path never calls it.

What it follows
  * Sec. 3.1, Eq. 1 (forward coupling):  Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2)):
    the queries come from the left stream, keys and values from the right stream.
  * Sec. 3.1, inverse pass:  X1 = Y1 - Attn(Norm(X1), Norm(X2), Norm(X2)) has X1 on both
    sides; it is solved by fixed-point iteration X1(i+1) = Y1 - Attn(Norm(X1(i)), ...),
    started from X1(0) = Y1, and the paper runs one iteration.  `inverse` takes the number
    of iterations, so the error the paper only asserts can be measured.
  * Sec. 3.2 (projection adapters):  Attn(a, b, b) = P_down(Attn_pt(P_up(a), P_up(b), P_up(b))),
    two bias-free linear maps d/2 -> d and d -> d/2; one P_up serves query, key and value.
  * Attn_pt: the paper only names it (the base model's self-attention, Sec. 3 intro).  The
    base model family fixes it: linear q/k/v projections with bias, rotary position
    embedding on q and k (pairs (i, i + hd/2) of a head rotated by pos * theta^(-2i/hd)),
    causal scaled-dot-product attention per head with scale hd^(-1/2), grouped key/value
    heads (n_kv_heads divides n_heads), and a bias-free output projection.
  * Norm: RMSNorm over the d/2-wide stream with one learnable scale that serves both
    streams (the base layer has one norm in front of its attention).
  * Backward (Sec. 2 "Reversible Networks", Sec. 3.1): the transpose-Jacobian of the same
    branch with respect to both streams and every weight.

Tokens are batch-major: token t = b * S + s is position s of sequence b; sequences do not
attend to each other.  All matrices are [out, in].

Weights (dict of arrays):
  norm_gamma [h] | w_up [d, h] | w_down [h, d] | w_q [d, d], b_q [d] |
  w_k [d_kv, d], b_k [d_kv] | w_v [d_kv, d], b_v [d_kv] | w_o [d, d]      (d_kv = n_kv_heads * hd)

Pins (tests/test_oracle_attn_pins.py): a loop-by-loop brute-force evaluation, the installed
base-model attention layer, causality, the uniform-attention closed form, the relative-
position property of the rotary embedding, central finite differences on every input and
weight, zero adapters, and convergence of the fixed-point inverse.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

F64 = np.float64


def _w(p: Dict[str, np.ndarray], name: str) -> np.ndarray:
    return np.asarray(p[name], dtype=F64)


# --------------------------------------------------------------------------- #
# Norm (Eq. 1: Norm(X1), Norm(X2))
# --------------------------------------------------------------------------- #
def norm_fwd(x: np.ndarray, gamma: Optional[np.ndarray], eps: float):
    """n = x * r * gamma with r = (mean(x^2) + eps)^-1/2 per token."""
    x = np.asarray(x, dtype=F64)
    r = 1.0 / np.sqrt(np.mean(x * x, axis=-1) + eps)
    n = x * r[..., None]
    if gamma is not None:
        n = n * np.asarray(gamma, dtype=F64)
    return n, r


def norm_bwd(x, gamma, r, dn):
    """Gradients of n = x * r * gamma: returns (dx, dgamma)."""
    x = np.asarray(x, dtype=F64)
    g = np.ones(x.shape[-1], dtype=F64) if gamma is None else np.asarray(gamma, dtype=F64)
    gdn = dn * g
    h = x.shape[-1]
    dx = r[:, None] * gdn - x * (r ** 3)[:, None] * (np.sum(gdn * x, axis=-1) / h)[:, None]
    dgamma = np.sum(dn * x * r[:, None], axis=0)
    return dx, dgamma


# --------------------------------------------------------------------------- #
# Rotary position embedding
# --------------------------------------------------------------------------- #
def rope_angles(S: int, hd: int, theta: float) -> np.ndarray:
    """angle[s, i] = s * theta^(-2i/hd), i < hd/2."""
    inv_freq = theta ** (-np.arange(0, hd, 2, dtype=F64) / hd)
    return np.arange(S, dtype=F64)[:, None] * inv_freq[None, :]


def rope_apply(x: np.ndarray, ang: np.ndarray, sign: float = 1.0) -> np.ndarray:
    """x [..., S, hd]: rotates each pair (x[i], x[i + hd/2]) by sign * ang[s, i]."""
    half = x.shape[-1] // 2
    c, s = np.cos(ang), np.sin(sign * ang)
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


# --------------------------------------------------------------------------- #
# Attn_pt(u_q, u_kv, u_kv)
# --------------------------------------------------------------------------- #
def _heads(x: np.ndarray, B: int, S: int, nh: int, hd: int) -> np.ndarray:
    """[B*S, nh*hd] -> [B, nh, S, hd]."""
    return x.reshape(B, S, nh, hd).transpose(0, 2, 1, 3)


def _unheads(x: np.ndarray) -> np.ndarray:
    """[B, nh, S, hd] -> [B*S, nh*hd]."""
    B, nh, S, hd = x.shape
    return x.transpose(0, 2, 1, 3).reshape(B * S, nh * hd)


def attn_pt(p, uq: np.ndarray, ukv: np.ndarray, S: int, n_heads: int, n_kv_heads: int,
            theta: float = 1e6, causal: bool = True):
    """The base model's attention with queries from uq and keys/values from ukv.
    Returns (a [T, d], cache of intermediates for the backward pass)."""
    T, d = uq.shape
    B = T // S
    assert B * S == T and d % n_heads == 0 and n_heads % n_kv_heads == 0
    hd = d // n_heads
    rep = n_heads // n_kv_heads
    q = uq @ _w(p, "w_q").T + _w(p, "b_q")
    k = ukv @ _w(p, "w_k").T + _w(p, "b_k")
    v = ukv @ _w(p, "w_v").T + _w(p, "b_v")
    ang = rope_angles(S, hd, theta)
    qh = rope_apply(_heads(q, B, S, n_heads, hd), ang)           # [B, nh, S, hd]
    kh = rope_apply(_heads(k, B, S, n_kv_heads, hd), ang)        # [B, nkv, S, hd]
    vh = _heads(v, B, S, n_kv_heads, hd)
    kx = np.repeat(kh, rep, axis=1)                              # query head j reads kv head j // rep
    vx = np.repeat(vh, rep, axis=1)
    sc = np.einsum("bhsd,bhtd->bhst", qh, kx) / np.sqrt(hd)
    if causal:
        mask = np.tril(np.ones((S, S), dtype=bool))
        sc = np.where(mask, sc, -np.inf)
    sc = sc - sc.max(axis=-1, keepdims=True)
    P = np.exp(sc)
    P = P / P.sum(axis=-1, keepdims=True)
    oh = np.einsum("bhst,bhtd->bhsd", P, vx)
    o = _unheads(oh)
    a = o @ _w(p, "w_o").T
    cache = dict(uq=uq, ukv=ukv, qh=qh, kx=kx, vx=vx, P=P, o=o, ang=ang, B=B, S=S, hd=hd, rep=rep)
    return a, cache


def attn_pt_bwd(p, cache, da: np.ndarray, n_heads: int, n_kv_heads: int):
    """Transpose-Jacobian of attn_pt.  Returns (duq, dukv, grads of w_q b_q w_k b_k w_v b_v w_o)."""
    B, S, hd, rep = cache["B"], cache["S"], cache["hd"], cache["rep"]
    P, qh, kx, vx, ang = cache["P"], cache["qh"], cache["kx"], cache["vx"], cache["ang"]
    g = {}
    g["w_o"] = da.T @ cache["o"]
    do = da @ _w(p, "w_o")
    doh = _heads(do, B, S, n_heads, hd)
    dvx = np.einsum("bhst,bhsd->bhtd", P, doh)
    dP = np.einsum("bhsd,bhtd->bhst", doh, vx)
    dS = P * (dP - np.sum(dP * P, axis=-1, keepdims=True))       # softmax backward, masked entries have P = 0
    dS = dS / np.sqrt(hd)
    dqh = np.einsum("bhst,bhtd->bhsd", dS, kx)
    dkx = np.einsum("bhst,bhsd->bhtd", dS, qh)
    # query heads that share a key/value head add their gradients
    dkh = dkx.reshape(B, n_kv_heads, rep, S, hd).sum(axis=2)
    dvh = dvx.reshape(B, n_kv_heads, rep, S, hd).sum(axis=2)
    # the rotation is orthogonal: its transpose rotates by the opposite angle
    dq = _unheads(rope_apply(dqh, ang, -1.0))
    dk = _unheads(rope_apply(dkh, ang, -1.0))
    dv = _unheads(dvh)
    uq, ukv = cache["uq"], cache["ukv"]
    g["w_q"], g["b_q"] = dq.T @ uq, dq.sum(axis=0)
    g["w_k"], g["b_k"] = dk.T @ ukv, dk.sum(axis=0)
    g["w_v"], g["b_v"] = dv.T @ ukv, dv.sum(axis=0)
    duq = dq @ _w(p, "w_q")
    dukv = dk @ _w(p, "w_k") + dv @ _w(p, "w_v")
    return duq, dukv, g


# --------------------------------------------------------------------------- #
# The branch A(X1, X2) = P_down(Attn_pt(P_up Norm(X1), P_up Norm(X2), P_up Norm(X2)))
# --------------------------------------------------------------------------- #
def branch(p, X1, X2, S: int, n_heads: int, n_kv_heads: int, eps: float = 1e-6, theta: float = 1e6,
           causal: bool = True):
    X1 = np.asarray(X1, dtype=F64)
    X2 = np.asarray(X2, dtype=F64)
    n1, r1 = norm_fwd(X1, p.get("norm_gamma"), eps)
    n2, r2 = norm_fwd(X2, p.get("norm_gamma"), eps)
    u1 = n1 @ _w(p, "w_up").T
    u2 = n2 @ _w(p, "w_up").T
    a, cache = attn_pt(p, u1, u2, S, n_heads, n_kv_heads, theta, causal)
    A = a @ _w(p, "w_down").T
    cache.update(X1=X1, X2=X2, n1=n1, n2=n2, r1=r1, r2=r2, a=a)
    return A, cache


def forward(p, X1, X2, S: int, n_heads: int, n_kv_heads: int, eps: float = 1e-6, theta: float = 1e6,
            causal: bool = True):
    """Eq. 1: Y1 = X1 + Attn(Norm(X1), Norm(X2), Norm(X2))."""
    A, _ = branch(p, X1, X2, S, n_heads, n_kv_heads, eps, theta, causal)
    return np.asarray(X1, dtype=F64) + A


def inverse(p, Y1, X2, S: int, n_heads: int, n_kv_heads: int, n_iter: int = 1, eps: float = 1e-6,
            theta: float = 1e6, causal: bool = True):
    """Sec. 3.1 inverse pass: n_iter fixed-point iterations started from X1 = Y1."""
    Y1 = np.asarray(Y1, dtype=F64)
    X1 = Y1.copy()
    for _ in range(int(n_iter)):
        A, _ = branch(p, X1, X2, S, n_heads, n_kv_heads, eps, theta, causal)
        X1 = Y1 - A
    return X1


def backward(p, X1, X2, dY1, S: int, n_heads: int, n_kv_heads: int, eps: float = 1e-6, theta: float = 1e6,
             causal: bool = True):
    """Gradients of <dY1, Y1> with Y1 = X1 + A(X1, X2).
    Returns (dX1, dX2, grads): dX1 includes the residual path (dY1 itself); dX2 is the branch's
    contribution through keys and values only."""
    dY1 = np.asarray(dY1, dtype=F64)
    _, c = branch(p, X1, X2, S, n_heads, n_kv_heads, eps, theta, causal)
    g = {}
    g["w_down"] = dY1.T @ c["a"]
    da = dY1 @ _w(p, "w_down")
    du1, du2, ga = attn_pt_bwd(p, c, da, n_heads, n_kv_heads)
    g.update(ga)
    g["w_up"] = du1.T @ c["n1"] + du2.T @ c["n2"]
    dn1 = du1 @ _w(p, "w_up")
    dn2 = du2 @ _w(p, "w_up")
    dx1, dg1 = norm_bwd(c["X1"], p.get("norm_gamma"), c["r1"], dn1)
    dx2, dg2 = norm_bwd(c["X2"], p.get("norm_gamma"), c["r2"], dn2)
    g["norm_gamma"] = dg1 + dg2
    return dY1 + dx1, dx2, g
