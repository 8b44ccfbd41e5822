"""CPU oracle for the MoE coupling branch of a RevFFN block.  TEST INFRASTRUCTURE.

Plain numpy, fp64, slow on purpose: it writes out the definition of the branch
so that a reader can check it against the paper by eye.  It shares no code with
the CUDA library and is imported only by the tests, the smoke check and the
benchmark's CPU-baseline leg; the product path never calls it.

What it follows
  * Sec. 3.1, Eq. 2 (forward coupling):  Y2 = X2 + MLP(Norm(Y1)).
  * Sec. 3.1, inverse pass:              X2 = Y2 - MLP(Norm(Y1)).
  * Sec. 3.2 (projection adapters):      MLP(y) = P_down(MLP_pt(P_up(y))), two
    bias-free linear maps d/2 -> d and d -> d/2.
  * MLP_pt: the paper only names it (the base model's sparse MoE block, Sec. 3
    intro and Sec. 3.2 "Advantages").  The benchmark configurations fix it: a
    linear router, top-k selection, softmax over the k selected logits (gate
    weights sum to 1), routed SwiGLU experts, and a SwiGLU shared expert scaled
    by a sigmoid gate.  No token dropping, no biases in the experts.  A second gating
    mode ("softmax_all") takes the selected probabilities of a softmax over all E
    logits without renormalising them.
  * Norm: RMSNorm over the d/2-wide stream (the base model family's norm) with a
    learnable scale; "none" is available for tests.
  * Backward (Sec. 2 "Reversible Networks", Sec. 3.1): the transpose-Jacobian of
    the same branch, with the selected expert set held constant (top-k is
    piecewise constant).  Routers may be frozen (Sec. 3.3) but the gradient
    still flows through the gate values to the stream.

Pins (tests/test_oracle_*.py): exact invertibility in fp64, central finite
differences on every input and weight, gate sums, closed forms for E=1 / k=E /
identical experts / zero adapters, token-permutation equivariance, brute-force
top-k, and a library cross-check of MLP_pt.  The paper prints no worked
numeric example, so absolute output values have no printed golden to match.

Notation: T tokens, d model width, h = d/2 stream width, E experts, k top-k,
I expert intermediate, I_s shared intermediate.  All matrices are [out, in].
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

F64 = np.float64


def _w(p: Dict[str, np.ndarray], name: str, e: Optional[int] = None) -> np.ndarray:
    """A weight (or one expert's slice of it) widened to fp64."""
    a = p[name] if e is None else p[name][e]
    return np.asarray(a, dtype=F64)


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def silu(x):
    return x * sigmoid(x)


def has_shared(p) -> bool:
    return p.get("ws_gate") is not None


# --------------------------------------------------------------------------- #
# Norm (Eq. 2: Norm(Y1))
# --------------------------------------------------------------------------- #
def norm_fwd(y: np.ndarray, gamma: Optional[np.ndarray], eps: float, kind: str = "rms"):
    """n = y * r * gamma with r = (mean(y^2) + eps)^-1/2 per token (RMSNorm)."""
    y = np.asarray(y, dtype=F64)
    if kind == "none":
        return y.copy(), np.ones(y.shape[:-1], dtype=F64)
    r = 1.0 / np.sqrt(np.mean(y * y, axis=-1) + eps)
    n = y * r[..., None]
    if gamma is not None:
        n = n * np.asarray(gamma, dtype=F64)
    return n, r


# --------------------------------------------------------------------------- #
# Routing (MLP_pt, steps: logits -> top-k -> softmax over the selected k)
# --------------------------------------------------------------------------- #
def router_logits(u: np.ndarray, p) -> np.ndarray:
    L = u @ _w(p, "w_router").T
    if p.get("b_router") is not None:
        L = L + _w(p, "b_router")
    return L


def topk_indices(L: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest logits per row, by descending value; equal
    values go to the lower expert index first (stable sort of the negation)."""
    return np.argsort(-L, axis=-1, kind="stable")[..., :k]


def topk_margin(L: np.ndarray, k: int) -> np.ndarray:
    """Gap between the k-th and (k+1)-th largest logit per row (inf if k == E)."""
    if k >= L.shape[-1]:
        return np.full(L.shape[:-1], np.inf)
    s = -np.sort(-L, axis=-1)
    return s[..., k - 1] - s[..., k]


GATINGS = ("renorm", "softmax_all")


def gate_weights(L: np.ndarray, idx: np.ndarray, gating: str = "renorm") -> np.ndarray:
    """Gate weights of the selected experts.
      "renorm":      softmax over the selected logits only, so the k weights sum to 1
                     (what the benchmark definition asks for);
      "softmax_all": softmax over all E logits, the selected probabilities taken as
                     they are (they sum to less than 1 unless k == E): the variant in
                     which the top-k probabilities are not renormalised."""
    assert gating in GATINGS
    sel = np.take_along_axis(L, idx, axis=-1)
    if gating == "renorm":
        m = sel.max(axis=-1, keepdims=True)
        ex = np.exp(sel - m)
        return ex / ex.sum(axis=-1, keepdims=True)
    m = L.max(axis=-1, keepdims=True)
    return np.exp(sel - m) / np.exp(L - m).sum(axis=-1, keepdims=True)


# --------------------------------------------------------------------------- #
# FP8 variant of the routed experts (not in the paper: a variant of MLP_pt's arithmetic in
# which the routed experts' three products take e4m3 operands, each row of an operand scaled
# by its own power-free fp32 factor).  The quantisation DECIDES integer codes, so it is
# written in the precision the kernels use: operands are first rounded to bf16 (what the
# kernels hold), the scale and the scaled value are fp32, the code is e4m3 by round to
# nearest even with saturation to the largest finite value.
# --------------------------------------------------------------------------- #
E4M3_MAX = 448.0


def round_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bf16 value (ties to even), returned as fp32."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def e4m3_round(v: np.ndarray) -> np.ndarray:
    """Nearest e4m3 value (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities; ties to the
    even mantissa; magnitudes beyond 448 saturate to 448), returned as fp32."""
    v = np.asarray(v, dtype=np.float32)
    a = np.abs(v).astype(np.float64)
    _, e = np.frexp(a)                       # a = m * 2^e with m in [0.5, 1)
    e = np.maximum(e - 1, -6)                # exponent of the leading bit; subnormals share the exponent -6
    step = np.ldexp(1.0, e - 3)              # spacing of e4m3 values in that binade
    q = np.rint(a / step) * step             # np.rint rounds halves to even
    q = np.minimum(q, E4M3_MAX)
    return (np.sign(v) * q).astype(np.float32)


def quantize_rows_e4m3(x: np.ndarray):
    """Per row: scale = max|x| / 448 (1 for an all-zero row), codes = e4m3_round(x * (1 / scale)), every
    operation a correctly rounded fp32 one (the kernels multiply by the row's reciprocal).
    Returns (the codes' values as fp32 [rows, cols] -- what the product sums --, scale [rows])."""
    x = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(x), axis=-1)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    inv = (np.float32(1.0) / scale).astype(np.float32)
    q = e4m3_round((x * inv[..., None]).astype(np.float32))
    return q, scale


def fp8_matmul(xq, xs, wq, ws):
    """(x W^T) with both operands quantised per row: the exact sum of products of the codes, then the two scales."""
    acc = xq.astype(F64) @ wq.astype(F64).T
    return acc * xs.astype(F64)[:, None] * ws.astype(F64)[None, :]


# --------------------------------------------------------------------------- #
# One token, written out step by step (the definition)
# --------------------------------------------------------------------------- #
def branch_token(p, y: np.ndarray, k: int, eps: float = 1e-6, norm: str = "rms",
                 idx_override: Optional[np.ndarray] = None, gating: str = "renorm"):
    """F = P_down(MLP_pt(P_up(Norm(y)))) for one token y (length h).

    Returns (F, idx, gates, margin).  idx_override forces the expert set (used
    for tokens whose top-k margin is below the comparison threshold)."""
    n, _ = norm_fwd(y, p.get("norm_gamma"), eps, norm)      # Norm(Y1)
    u = _w(p, "w_up") @ n                                   # P_up, Sec. 3.2
    L = router_logits(u[None, :], p)[0]                     # router
    idx = topk_indices(L, k) if idx_override is None else np.asarray(idx_override)
    g = gate_weights(L[None, :], idx[None, :], gating)[0]
    z = np.zeros_like(u)
    for s, e in enumerate(idx):                             # routed SwiGLU experts
        a = _w(p, "w_gate", e) @ u
        b = _w(p, "w_upx", e) @ u
        z += g[s] * (_w(p, "w_downx", e) @ (silu(a) * b))
    if has_shared(p):                                       # gated shared expert
        a = _w(p, "ws_gate") @ u
        b = _w(p, "ws_up") @ u
        sg = sigmoid(np.dot(_w(p, "ws_sgate"), u))
        z += sg * (_w(p, "ws_down") @ (silu(a) * b))
    F = _w(p, "w_down") @ z                                 # P_down, Sec. 3.2
    return F, idx, g, topk_margin(L[None, :], k)[0]


# --------------------------------------------------------------------------- #
# All tokens (same arithmetic, tokens grouped per expert so matmul can be used)
# --------------------------------------------------------------------------- #
def branch(p, Y1: np.ndarray, k: int, eps: float = 1e-6, norm: str = "rms",
           route_override: Optional[np.ndarray] = None, keep: bool = False, gating: str = "renorm",
           fp8_experts: bool = False):
    """F[T,h] = MLP(Norm(Y1)) for all tokens.  Returns (F, info); info holds the
    routing (idx, gates, margin, logits) and, with keep=True, the intermediates
    the backward pass needs.  fp8_experts: the routed experts' products take e4m3 operands
    (see quantize_rows_e4m3): u and g*H are rounded to bf16 and quantised per token row, the
    expert weights per output row; everything else is unchanged."""
    Y1 = np.asarray(Y1, dtype=F64)
    T = Y1.shape[0]
    n, r = norm_fwd(Y1, p.get("norm_gamma"), eps, norm)
    u = n @ _w(p, "w_up").T
    L = router_logits(u, p)
    idx = topk_indices(L, k) if route_override is None else np.asarray(route_override)
    g = gate_weights(L, idx, gating)
    E = p["w_router"].shape[0]
    d = u.shape[1]
    z = np.zeros((T, d), dtype=F64)
    per_expert = {}
    for e in range(E):
        toks, slots = np.nonzero(idx == e)
        if toks.size == 0:
            continue
        ue = u[toks]
        if fp8_experts:
            uq, us = quantize_rows_e4m3(round_bf16(ue.astype(np.float32)))
            a = fp8_matmul(uq, us, *quantize_rows_e4m3(np.asarray(p["w_gate"][e], np.float32)))
            b = fp8_matmul(uq, us, *quantize_rows_e4m3(np.asarray(p["w_upx"][e], np.float32)))
            # the gate weight goes onto H before it is rounded and quantised (as the kernels do)
            hg = round_bf16((g[toks, slots][:, None] * (silu(a) * b)).astype(np.float32))
            hq, hs = quantize_rows_e4m3(hg)
            z[toks] += fp8_matmul(hq, hs, *quantize_rows_e4m3(np.asarray(p["w_downx"][e], np.float32)))
            continue
        a = ue @ _w(p, "w_gate", e).T
        b = ue @ _w(p, "w_upx", e).T
        hm = silu(a) * b
        f = hm @ _w(p, "w_downx", e).T
        z[toks] += g[toks, slots][:, None] * f
        if keep:
            per_expert[e] = (toks, slots, a, b, hm, f)
    info = dict(idx=idx, gates=g, logits=L, margin=topk_margin(L, k))
    if has_shared(p):
        a_s = u @ _w(p, "ws_gate").T
        b_s = u @ _w(p, "ws_up").T
        h_s = silu(a_s) * b_s
        S = h_s @ _w(p, "ws_down").T
        sg = sigmoid(u @ _w(p, "ws_sgate"))
        z = z + sg[:, None] * S
        info["sgate"] = sg
        if keep:
            info.update(a_s=a_s, b_s=b_s, h_s=h_s, S=S)
    F = z @ _w(p, "w_down").T
    if keep:
        info.update(n=n, r=r, u=u, z=z, per_expert=per_expert)
    return F, info


def forward(p, Y1, X2, k: int, eps: float = 1e-6, norm: str = "rms", route_override=None, gating: str = "renorm",
            fp8_experts: bool = False):
    """Eq. 2: Y2 = X2 + MLP(Norm(Y1)).  Returns (Y2, info)."""
    F, info = branch(p, Y1, k, eps, norm, route_override, gating=gating, fp8_experts=fp8_experts)
    info["F"] = F
    return np.asarray(X2, dtype=F64) + F, info


def inverse(p, Y1, Y2, k: int, eps: float = 1e-6, norm: str = "rms", route_override=None, gating: str = "renorm",
            fp8_experts: bool = False):
    """Inverse pass of Sec. 3.1: X2 = Y2 - MLP(Norm(Y1)).  Returns (X2, info)."""
    F, info = branch(p, Y1, k, eps, norm, route_override, gating=gating, fp8_experts=fp8_experts)
    info["F"] = F
    return np.asarray(Y2, dtype=F64) - F, info


# --------------------------------------------------------------------------- #
# Backward: J^T dY2 for the stream Y1 and every weight
# --------------------------------------------------------------------------- #
def backward(p, Y1, dY2, k: int, eps: float = 1e-6, norm: str = "rms", route_override=None,
             gating: str = "renorm"):
    """Gradients of <dY2, Y2> through Eq. 2 with Y1 as the only kept input
    (intermediates are recomputed, as reversible back-propagation does).

    Returns a dict with dy1 (= J^T dY2 w.r.t. Y1; the caller adds it to the
    gradient Y1 already carries), dx2 (= dY2) and one entry per weight."""
    Y1 = np.asarray(Y1, dtype=F64)
    G = np.asarray(dY2, dtype=F64)
    F, c = branch(p, Y1, k, eps, norm, route_override, keep=True, gating=gating)
    idx, g, u, n, r, z = c["idx"], c["gates"], c["u"], c["n"], c["r"], c["z"]
    T, h = Y1.shape
    E = p["w_router"].shape[0]
    out: Dict[str, np.ndarray] = {"dx2": G.copy(), "F": F, "idx": idx}

    # P_down:  F = z W_down^T
    dz = G @ _w(p, "w_down")
    out["w_down"] = G.T @ z
    du = np.zeros_like(u)

    # shared expert:  z += sg * S,  S = h_s Ws_d^T,  h_s = silu(a_s) * b_s
    if has_shared(p):
        sg, a_s, b_s, h_s, S = c["sgate"], c["a_s"], c["b_s"], c["h_s"], c["S"]
        dsg = np.sum(dz * S, axis=1)
        dS = sg[:, None] * dz
        dh = dS @ _w(p, "ws_down")
        out["ws_down"] = dS.T @ h_s
        s = sigmoid(a_s)
        da = dh * b_s * (s * (1.0 + a_s * (1.0 - s)))
        db = dh * (a_s * s)
        du += da @ _w(p, "ws_gate") + db @ _w(p, "ws_up")
        out["ws_gate"] = da.T @ u
        out["ws_up"] = db.T @ u
        dl = dsg * sg * (1.0 - sg)
        out["ws_sgate"] = dl @ u
        du += dl[:, None] * _w(p, "ws_sgate")[None, :]

    # routed experts:  z[t] += g[t,s] * f_e(u[t])
    dgate = np.zeros_like(g)
    out["w_gate"] = np.zeros(p["w_gate"].shape, dtype=F64)
    out["w_upx"] = np.zeros(p["w_upx"].shape, dtype=F64)
    out["w_downx"] = np.zeros(p["w_downx"].shape, dtype=F64)
    for e, (toks, slots, a, b, hm, f) in c["per_expert"].items():
        dze = dz[toks]
        dgate[toks, slots] = np.sum(dze * f, axis=1)
        df = g[toks, slots][:, None] * dze
        dh = df @ _w(p, "w_downx", e)
        out["w_downx"][e] = df.T @ hm
        s = sigmoid(a)
        da = dh * b * (s * (1.0 + a * (1.0 - s)))
        db = dh * (a * s)
        du[toks] += da @ _w(p, "w_gate", e) + db @ _w(p, "w_upx", e)
        out["w_gate"][e] = da.T @ u[toks]
        out["w_upx"][e] = db.T @ u[toks]

    # gates; the selection itself has zero gradient
    if gating == "renorm":
        # softmax over the selected logits: only those logits receive a gradient
        dsel = g * (dgate - np.sum(g * dgate, axis=1, keepdims=True))
        dL = np.zeros((T, E), dtype=F64)
        np.put_along_axis(dL, idx, dsel, axis=1)
    else:
        # softmax over all logits, g_s = p_s for the selected s:
        # dL_j = p_j ([j selected] dg_j - sum_s p_s dg_s) for every j
        L = c["logits"]
        prob = np.exp(L - L.max(axis=1, keepdims=True))
        prob = prob / prob.sum(axis=1, keepdims=True)
        dfull = np.zeros((T, E), dtype=F64)
        np.put_along_axis(dfull, idx, dgate, axis=1)
        dL = prob * (dfull - np.sum(g * dgate, axis=1, keepdims=True))
    out["w_router"] = dL.T @ u
    out["b_router"] = dL.sum(axis=0)
    du += dL @ _w(p, "w_router")

    # P_up:  u = n W_up^T
    dn = du @ _w(p, "w_up")
    out["w_up"] = du.T @ n

    # Norm:  n = y * r * gamma
    if norm == "none":
        out["dy1"] = dn
        out["norm_gamma"] = np.zeros(h, dtype=F64)
    else:
        gam = _w(p, "norm_gamma") if p.get("norm_gamma") is not None else np.ones(h, dtype=F64)
        q = dn * gam
        out["dy1"] = r[:, None] * q - Y1 * (r ** 3 * np.sum(q * Y1, axis=1) / h)[:, None]
        out["norm_gamma"] = np.sum(dn * Y1 * r[:, None], axis=0)
    return out


# --------------------------------------------------------------------------- #
# One optimiser step on the gradients above (Sec. 3.3 trains the adapters, then adapters
# and experts, with a first-order optimiser; plain SGD is the step written out here).
# --------------------------------------------------------------------------- #
def sgd_step(p, grads, lr: float, names):
    """W <- W - lr * dL/dW for the named weights (fp64); the others are returned as they are."""
    out = dict(p)
    for n in names:
        out[n] = _w(p, n) - lr * np.asarray(grads[n], dtype=F64)
    return out


def adam_step(p, grads, mom, var, lr: float, step: int, names, beta1: float = 0.9, beta2: float = 0.999,
              eps: float = 1e-8, weight_decay: float = 0.0):
    """One Adam step with decoupled weight decay on the named weights (fp64), written out from the rule's
    definition: m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;  m^ = m / (1 - b1^t);  v^ = v / (1 - b2^t);
    W <- W - lr (m^ / (sqrt(v^) + eps) + weight_decay W).  mom / var: dicts of the moment estimates before the
    step (missing = zeros).  Returns (weights, mom, var) after it.  (The paper names no optimiser for its method:
    this is the moment-based reading of the fused update, beside sgd_step.)"""
    out, m_out, v_out = dict(p), dict(mom), dict(var)
    for n in names:
        g = np.asarray(grads[n], dtype=F64)
        w = _w(p, n)
        m = beta1 * np.asarray(mom.get(n, 0.0), dtype=F64) + (1.0 - beta1) * g
        v = beta2 * np.asarray(var.get(n, 0.0), dtype=F64) + (1.0 - beta2) * g * g
        m_hat = m / (1.0 - beta1 ** step)
        v_hat = v / (1.0 - beta2 ** step)
        out[n] = w - lr * (m_hat / (np.sqrt(v_hat) + eps) + weight_decay * w)
        m_out[n], v_out[n] = m, v
    return out, m_out, v_out


# --------------------------------------------------------------------------- #
# A stack of coupling branches (Sec. 3.1: the two output streams of a layer are
# the input of the next one; Sec. 2: inputs are rebuilt layer by layer from the
# outputs during back-propagation, nothing is cached).
#
# Only the MoE branch of each block is modelled, so the streams swap roles from
# one layer to the next: layer l reads stream P_l and updates stream R_l,
# (P_l, R_l) = (A, B) for even l and (B, A) for odd l.  Both streams are
# therefore rewritten every two layers and reconstruction error compounds
# through both, as it does in the full block.
# --------------------------------------------------------------------------- #
def stack_forward(blocks, A, B, k: int, eps: float = 1e-6, norm: str = "rms", route_overrides=None,
                  gating: str = "renorm"):
    """R_l <- R_l + MLP_l(Norm(P_l)) for l = 0 .. L-1 (Eq. 2 per layer).
    Returns (A, B, infos); infos[l] is the layer's `forward` info."""
    A = np.array(A, dtype=F64)
    B = np.array(B, dtype=F64)
    infos = []
    for l, p in enumerate(blocks):
        ro = None if route_overrides is None else route_overrides[l]
        if l % 2 == 0:
            B, info = forward(p, A, B, k, eps, norm, ro, gating)
        else:
            A, info = forward(p, B, A, k, eps, norm, ro, gating)
        infos.append(info)
    return A, B, infos


def stack_inverse(blocks, A, B, k: int, eps: float = 1e-6, norm: str = "rms", route_overrides=None,
                  gating: str = "renorm"):
    """Undo `stack_forward` from its outputs: R_l <- R_l - MLP_l(Norm(P_l)) for
    l = L-1 .. 0 (inverse pass of Sec. 3.1 per layer).  Returns (A, B)."""
    A = np.array(A, dtype=F64)
    B = np.array(B, dtype=F64)
    for l in reversed(range(len(blocks))):
        ro = None if route_overrides is None else route_overrides[l]
        if l % 2 == 0:
            B, _ = inverse(blocks[l], A, B, k, eps, norm, ro, gating)
        else:
            A, _ = inverse(blocks[l], B, A, k, eps, norm, ro, gating)
    return A, B


def stack_backward(blocks, A_out, B_out, gA, gB, k: int, eps: float = 1e-6, norm: str = "rms",
                   route_overrides=None, gating: str = "renorm"):
    """Reversible back-propagation through the stack: for l = L-1 .. 0 rebuild
    the layer's input from its output, then push the gradient through the
    layer (dP += J^T dR, dR passes through unchanged).

    A_out, B_out: outputs of `stack_forward`; gA, gB: dLoss/dA_out, dLoss/dB_out.
    Returns (A_in, B_in, dA_in, dB_in, grads); grads[l] holds layer l's weight
    gradients (the dict `backward` returns)."""
    A = np.array(A_out, dtype=F64)
    B = np.array(B_out, dtype=F64)
    gA = np.array(gA, dtype=F64)
    gB = np.array(gB, dtype=F64)
    grads = [None] * len(blocks)
    for l in reversed(range(len(blocks))):
        ro = None if route_overrides is None else route_overrides[l]
        p = blocks[l]
        if l % 2 == 0:
            B, _ = inverse(p, A, B, k, eps, norm, ro, gating)
            g = backward(p, A, gB, k, eps, norm, ro, gating)
            gA = gA + g["dy1"]
        else:
            A, _ = inverse(p, B, A, k, eps, norm, ro, gating)
            g = backward(p, B, gA, k, eps, norm, ro, gating)
            gB = gB + g["dy1"]
        grads[l] = g
    return A, B, gA, gB, grads
