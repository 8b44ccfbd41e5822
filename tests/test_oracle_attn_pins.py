"""Pins for the attention-branch oracle: each test checks it against something the paper or the
mathematics fixes, not against itself (Sec. 3.1 Eq. 1 and inverse pass, Sec. 3.2 adapters)."""
import math

import numpy as np
import pytest
import torch

from oracle import revffn_attn_oracle as orc

H, D, NH, NKV, S, B = 8, 16, 4, 2, 6, 2          # stream width, model width, heads, kv heads, seq, batch
HD = D // NH
THETA = 100.0


def _weights(seed=0, std=0.3, d=D, h=H, nh=NH, nkv=NKV):
    rng = np.random.default_rng(seed)
    dkv = nkv * (d // nh)
    n = lambda *s: rng.standard_normal(s) * std
    return {
        "norm_gamma": 1.0 + 0.1 * rng.standard_normal(h),
        "w_up": n(d, h), "w_down": n(h, d), "w_q": n(d, d), "b_q": n(d), "w_k": n(dkv, d), "b_k": n(dkv),
        "w_v": n(dkv, d), "b_v": n(dkv), "w_o": n(d, d),
    }


def _streams(seed=1, T=B * S, h=H):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((T, h)), rng.standard_normal((T, h)), rng.standard_normal((T, h))


# ------------------------------------------------------------------ brute force, loop by loop
def _brute_forward(p, X1, X2, S, nh, nkv, eps, theta):
    """Eq. 1 evaluated scalar by scalar with Python loops (no shared helper with the oracle)."""
    T, h = X1.shape
    d = p["w_up"].shape[0]
    hd = d // nh
    rep = nh // nkv

    def norm(x):
        out = np.zeros_like(x)
        for t in range(T):
            ms = sum(x[t, i] ** 2 for i in range(h)) / h
            for i in range(h):
                out[t, i] = x[t, i] / math.sqrt(ms + eps) * p["norm_gamma"][i]
        return out

    def lin(x, w, b=None):
        out = np.zeros((x.shape[0], w.shape[0]))
        for t in range(x.shape[0]):
            for o in range(w.shape[0]):
                out[t, o] = sum(x[t, i] * w[o, i] for i in range(w.shape[1])) + (0.0 if b is None else b[o])
        return out

    def rot(vec, pos):
        out = np.zeros(hd)
        for i in range(hd // 2):
            ang = pos * theta ** (-2.0 * i / hd)
            out[i] = vec[i] * math.cos(ang) - vec[i + hd // 2] * math.sin(ang)
            out[i + hd // 2] = vec[i + hd // 2] * math.cos(ang) + vec[i] * math.sin(ang)
        return out

    u1, u2 = lin(norm(X1), p["w_up"]), lin(norm(X2), p["w_up"])
    q, k, v = lin(u1, p["w_q"], p["b_q"]), lin(u2, p["w_k"], p["b_k"]), lin(u2, p["w_v"], p["b_v"])
    o = np.zeros((T, d))
    for b in range(T // S):
        for hq in range(nh):
            hk = hq // rep
            for s in range(S):
                qv = rot(q[b * S + s, hq * hd:(hq + 1) * hd], s)
                logits = []
                for j in range(s + 1):                                  # causal: keys 0..s
                    kv = rot(k[b * S + j, hk * hd:(hk + 1) * hd], j)
                    logits.append(sum(qv[i] * kv[i] for i in range(hd)) / math.sqrt(hd))
                m = max(logits)
                w = [math.exp(x - m) for x in logits]
                z = sum(w)
                for j in range(s + 1):
                    o[b * S + s, hq * hd:(hq + 1) * hd] += w[j] / z * v[b * S + j, hk * hd:(hk + 1) * hd]
    return X1 + lin(lin(o, p["w_o"]), p["w_down"])


def test_forward_matches_a_scalar_loop_evaluation():
    p = _weights(3)
    X1, X2, _ = _streams(4)
    Y = orc.forward(p, X1, X2, S, NH, NKV, eps=1e-6, theta=THETA)
    ref = _brute_forward(p, X1, X2, S, NH, NKV, 1e-6, THETA)
    assert np.allclose(Y, ref, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ library cross-check of Attn_pt
def test_attn_pt_matches_the_installed_base_model_attention():
    m = pytest.importorskip("transformers.models.qwen2_moe.modeling_qwen2_moe")
    p = _weights(5)
    try:
        cfg = m.Qwen2MoeConfig(hidden_size=D, num_attention_heads=NH, num_key_value_heads=NKV, rope_theta=THETA,
                               num_hidden_layers=1, max_position_embeddings=64)
        cfg._attn_implementation = "eager"
        att = m.Qwen2MoeAttention(cfg, 0).double()
        rot = m.Qwen2MoeRotaryEmbedding(cfg)
        T = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
        new = {"q_proj.weight": T(p["w_q"]), "q_proj.bias": T(p["b_q"]), "k_proj.weight": T(p["w_k"]),
               "k_proj.bias": T(p["b_k"]), "v_proj.weight": T(p["w_v"]), "v_proj.bias": T(p["b_v"]),
               "o_proj.weight": T(p["w_o"])}
        sd = att.state_dict()
        if set(new) != set(sd) or any(new[k].shape != sd[k].shape for k in new):
            pytest.skip("installed transformers lays the layer out differently")
        att.load_state_dict(new)
        u = np.random.default_rng(6).standard_normal((B * S, D))
        x = torch.tensor(u).reshape(B, S, D)
        pos = torch.arange(S)[None].expand(B, -1)
        cos, sin = rot(x, pos)
        mask = torch.full((S, S), float("-inf"), dtype=torch.float64).triu(1)[None, None].expand(B, 1, S, S)
        with torch.no_grad():
            ref, _ = att(x, position_embeddings=(cos.double(), sin.double()), attention_mask=mask)
    except (TypeError, AttributeError) as exc:      # API drift in the library
        pytest.skip(f"transformers API differs: {exc}")
    # the library is a self-attention layer: same input on the query and the key/value side
    a, _ = orc.attn_pt(p, u, u, S, NH, NKV, theta=THETA)
    # the library builds its cos/sin tables in fp32
    assert np.allclose(a, ref.reshape(B * S, D).numpy(), rtol=1e-5, atol=1e-6)


# ------------------------------------------------------------------ structure of the attention
def test_causality_and_batch_independence():
    p = _weights(7)
    X1, X2, _ = _streams(8)
    Y = orc.forward(p, X1, X2, S, NH, NKV, theta=THETA)
    X1b, X2b = X1.copy(), X2.copy()
    s0 = 3
    X2b[s0:S] += 1.0                                 # sequence 0, positions >= s0, key/value side
    X1b[S + s0] -= 2.0                               # sequence 1, one query position
    Yb = orc.forward(p, X1b, X2b, S, NH, NKV, theta=THETA)
    assert np.array_equal(Y[:s0], Yb[:s0])           # earlier positions of sequence 0 see nothing of it
    assert not np.allclose(Y[s0:S], Yb[s0:S])
    changed = np.any(Y[S:] != Yb[S:], axis=1)        # in sequence 1 only the perturbed query row moves
    assert changed.tolist() == [i == s0 for i in range(S)]


def test_uniform_attention_closed_form():
    """Without key projection every logit is 0, so position s averages the values of positions 0..s."""
    p = _weights(9)
    p["w_k"] = np.zeros_like(p["w_k"]); p["b_k"] = np.zeros_like(p["b_k"])
    X1, X2, _ = _streams(10)
    n2 = X2 / np.sqrt((X2 ** 2).mean(axis=1, keepdims=True) + 1e-6) * p["norm_gamma"]
    v = n2 @ p["w_up"].T @ p["w_v"].T + p["b_v"]                       # [T, d_kv]
    rep = NH // NKV
    o = np.zeros((B * S, D))
    for b in range(B):
        run = np.cumsum(v[b * S:(b + 1) * S], axis=0) / np.arange(1, S + 1)[:, None]
        for hq in range(NH):
            o[b * S:(b + 1) * S, hq * HD:(hq + 1) * HD] = run[:, (hq // rep) * HD:(hq // rep + 1) * HD]
    ref = X1 + o @ p["w_o"].T @ p["w_down"].T
    assert np.allclose(orc.forward(p, X1, X2, S, NH, NKV, theta=THETA), ref, rtol=1e-12, atol=1e-13)


def test_rotary_embedding_depends_on_relative_position_only():
    rng = np.random.default_rng(11)
    q, k = rng.standard_normal(HD), rng.standard_normal(HD)
    ang = orc.rope_angles(S, HD, THETA)
    Q = orc.rope_apply(np.tile(q, (S, 1)), ang)
    K = orc.rope_apply(np.tile(k, (S, 1)), ang)
    G = Q @ K.T
    # <R(s) q, R(j) k> is a function of s - j: the Gram matrix is constant along its diagonals
    for off in range(-(S - 1), S):
        diag = np.diagonal(G, offset=off)
        assert np.allclose(diag, diag[0], rtol=1e-12, atol=1e-13)
    assert np.allclose(np.linalg.norm(Q, axis=1), np.linalg.norm(q))      # a rotation keeps the length
    assert np.allclose(Q[0], q) and np.allclose(K[0], k)                  # position 0 is not rotated
    # first pair at position 1 turns by exactly 1 radian (i = 0: theta^0)
    a, b = q[0], q[HD // 2]
    assert np.allclose([Q[1, 0], Q[1, HD // 2]], [a * math.cos(1) - b * math.sin(1), b * math.cos(1) + a * math.sin(1)])
    # undoing the rotation
    assert np.allclose(orc.rope_apply(Q, ang, -1.0), np.tile(q, (S, 1)))


def test_attention_weights_are_a_causal_distribution():
    p = _weights(12)
    X1, X2, _ = _streams(13)
    _, c = orc.branch(p, X1, X2, S, NH, NKV, theta=THETA)
    P = c["P"]
    assert P.shape == (B, NH, S, S)
    assert np.allclose(P.sum(axis=-1), 1.0, rtol=1e-14)
    assert np.all(P >= 0) and np.all(np.triu(P, 1) == 0)
    assert np.allclose(P[:, :, 0, 0], 1.0)                    # the first position can only see itself


def test_zero_adapters_make_the_block_the_identity():
    p = _weights(14)
    X1, X2, dY = _streams(15)
    q = dict(p); q["w_down"] = np.zeros_like(p["w_down"])
    assert np.array_equal(orc.forward(q, X1, X2, S, NH, NKV, theta=THETA), X1)
    assert np.array_equal(orc.inverse(q, X1, X2, S, NH, NKV, n_iter=1, theta=THETA), X1)
    dX1, dX2, g = orc.backward(q, X1, X2, dY, S, NH, NKV, theta=THETA)
    assert np.array_equal(dX1, dY) and not dX2.any()
    assert g["w_down"].any() and not g["w_up"].any() and not g["w_q"].any()


# ------------------------------------------------------------------ inverse pass (Sec. 3.1)
def test_fixed_point_inverse_converges_to_the_input():
    p = _weights(16, std=0.12)                                # small weights: the branch is a contraction
    X1, X2, _ = _streams(17)
    Y1 = orc.forward(p, X1, X2, S, NH, NKV, theta=THETA)
    errs = [np.linalg.norm(orc.inverse(p, Y1, X2, S, NH, NKV, n_iter=n, theta=THETA) - X1) / np.linalg.norm(X1)
            for n in (0, 1, 2, 4, 8, 40)]
    assert errs[0] > 1e-4                                     # Y1 itself is not X1
    assert all(b < 0.5 * a for a, b in zip(errs[:5], errs[1:5]))      # geometric decrease
    assert errs[-1] < 1e-10                                   # exact invertibility in fp64
    # one iteration is by definition Y1 - Attn evaluated at Norm(Y1) on the query side
    A0, _ = orc.branch(p, Y1, X2, S, NH, NKV, theta=THETA)
    assert np.array_equal(orc.inverse(p, Y1, X2, S, NH, NKV, n_iter=1, theta=THETA), Y1 - A0)
    # a fixed point of the iteration solves the equation of the inverse pass
    Xs = orc.inverse(p, Y1, X2, S, NH, NKV, n_iter=60, theta=THETA)
    As, _ = orc.branch(p, Xs, X2, S, NH, NKV, theta=THETA)
    assert np.allclose(Xs + As, Y1, rtol=1e-13, atol=1e-13)


# ------------------------------------------------------------------ backward: central differences
def _loss(p, X1, X2, dY):
    return float(np.sum(orc.forward(p, X1, X2, S, NH, NKV, theta=THETA) * dY))


def test_backward_matches_central_differences_on_streams_and_weights():
    p = _weights(18)
    X1, X2, dY = _streams(19)
    dX1, dX2, g = orc.backward(p, X1, X2, dY, S, NH, NKV, theta=THETA)
    rng = np.random.default_rng(20)
    eps = 1e-6

    def fd(arr, idx, f):
        old = arr[idx]
        arr[idx] = old + eps; up = f()
        arr[idx] = old - eps; dn = f()
        arr[idx] = old
        return (up - dn) / (2 * eps)

    for name, grad, arr in (("X1", dX1, X1), ("X2", dX2, X2)):
        for _ in range(6):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            num = fd(arr, idx, lambda: _loss(p, X1, X2, dY))
            assert abs(num - grad[idx]) <= 1e-6 * max(1.0, abs(num)), (name, idx, num, grad[idx])
    assert set(g) == set(p)
    for name in p:
        for _ in range(5):
            idx = tuple(rng.integers(0, s) for s in p[name].shape)
            num = fd(p[name], idx, lambda: _loss(p, X1, X2, dY))
            assert abs(num - g[name][idx]) <= 1e-6 * max(1.0, abs(num)), (name, idx, num, g[name][idx])


def test_key_value_heads_shared_by_a_group_equal_replicated_heads():
    """Grouped key/value heads are the same function as full heads whose weights repeat."""
    p = _weights(21)
    X1, X2, dY = _streams(22)
    rep = NH // NKV
    q = dict(p)
    for w, b in (("w_k", "b_k"), ("w_v", "b_v")):
        q[w] = np.repeat(p[w].reshape(NKV, HD, D), rep, axis=0).reshape(NH * HD, D)
        q[b] = np.repeat(p[b].reshape(NKV, HD), rep, axis=0).reshape(NH * HD)
    Y_g = orc.forward(p, X1, X2, S, NH, NKV, theta=THETA)
    Y_f = orc.forward(q, X1, X2, S, NH, NH, theta=THETA)
    assert np.allclose(Y_g, Y_f, rtol=1e-13, atol=1e-14)
    _, dX2_g, g_g = orc.backward(p, X1, X2, dY, S, NH, NKV, theta=THETA)
    _, dX2_f, g_f = orc.backward(q, X1, X2, dY, S, NH, NH, theta=THETA)
    assert np.allclose(dX2_g, dX2_f, rtol=1e-12, atol=1e-13)
    assert np.allclose(g_g["w_k"], g_f["w_k"].reshape(NKV, rep, HD, D).sum(axis=1).reshape(NKV * HD, D), rtol=1e-12)
