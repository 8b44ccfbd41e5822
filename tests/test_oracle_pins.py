"""Pins for the CPU oracle: what the paper and the mathematics fix, checked
against something other than the oracle's own formulas.

The paper prints no worked numeric example, so the pins are: exact
invertibility (Sec. 3.1), finite differences of the forward map, gate sums,
special cases that collapse to textbook forms, brute force on tiny inputs, an
independently written torch composite with autograd, and a library call to the
installed Qwen2-MoE sparse block for MLP_pt.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights

TINY = BlockConfig("tiny", tokens=7, d_model=16, n_experts=5, top_k=2, d_expert=12,
                   d_shared=10, weight_dtype="f32")


def _tiny(seed=0, scale=8.0, **kw):
    """Tiny block with weights scaled up so that every term matters."""
    cfg = BlockConfig(**{**TINY.__dict__, **kw})
    p = make_weights(cfg, seed)
    for name in p:
        if name != "norm_gamma":
            p[name] = p[name] * scale
    s = make_streams(cfg, seed)
    return cfg, p, s


# ------------------------------------------------------------------ invertibility
def test_invertible_fp64_c0():
    cfg = CONFIGS["C0"]
    p, s = make_weights(cfg, 0), make_streams(cfg, 0)
    y2, _ = orc.forward(p, s["y1"], s["x2"], cfg.top_k, cfg.norm_eps)
    x2, _ = orc.inverse(p, s["y1"], y2, cfg.top_k, cfg.norm_eps)
    assert np.max(np.abs(x2 - s["x2"].astype(np.float64))) <= 1e-10


def test_forward_is_coupling_add():
    cfg, p, s = _tiny()
    y2, info = orc.forward(p, s["y1"], s["x2"], cfg.top_k)
    assert np.allclose(y2 - s["x2"], info["F"], rtol=0, atol=1e-14)
    assert np.abs(info["F"]).max() > 1e-3      # the branch is not trivially zero


# ------------------------------------------------------------------ routing
def test_gates_sum_to_one_and_positive():
    cfg = CONFIGS["C0"]
    p, s = make_weights(cfg, 0), make_streams(cfg, 0)
    _, info = orc.forward(p, s["y1"], s["x2"], cfg.top_k)
    g = info["gates"]
    assert g.shape == (cfg.tokens, cfg.top_k)
    assert np.allclose(g.sum(axis=1), 1.0, atol=1e-14)
    assert (g > 0).all() and (g <= 1).all()
    # gates are ordered like their logits: descending
    assert (np.diff(g, axis=1) <= 1e-15).all()


def test_topk_brute_force_and_ties():
    rng = np.random.default_rng(1)
    L = rng.standard_normal((40, 6))
    L[3, 1] = L[3, 4] = L[3].max() + 1.0           # tie for the top place
    L[5, :] = 0.25                                   # all equal
    L[7, 2] = L[7, 5] = np.sort(L[7])[-2]          # tie straddling the k boundary region
    for k in (1, 2, 3, 6):
        idx = orc.topk_indices(L, k)
        for t in range(L.shape[0]):
            # brute force: best k-subset by (sum of logits), ties -> lexicographically lowest indices
            order = sorted(range(6), key=lambda e: (-L[t, e], e))[:k]
            assert list(idx[t]) == order
    assert list(orc.topk_indices(L, 2)[3]) == [1, 4]
    assert list(orc.topk_indices(L, 3)[5]) == [0, 1, 2]


def test_margin_matches_sorted_gap():
    rng = np.random.default_rng(2)
    L = rng.standard_normal((10, 8))
    m = orc.topk_margin(L, 3)
    for t in range(10):
        s = sorted(L[t], reverse=True)
        assert m[t] == pytest.approx(s[2] - s[3])
    assert np.isinf(orc.topk_margin(L, 8)).all()


# ------------------------------------------------------------------ per-token definition == batched
def test_token_definition_matches_batched():
    cfg, p, s = _tiny(3)
    F, info = orc.branch(p, s["y1"], cfg.top_k)
    for t in range(cfg.tokens):
        Ft, idx, g, margin = orc.branch_token(p, s["y1"][t], cfg.top_k)
        assert list(idx) == list(info["idx"][t])
        assert np.allclose(g, info["gates"][t], atol=1e-14)
        assert np.allclose(Ft, F[t], rtol=1e-12, atol=1e-14)
        assert margin == pytest.approx(info["margin"][t])


# ------------------------------------------------------------------ independent torch composite
def _torch_branch(p, y1, k, eps=1e-6, norm="rms"):
    """Dense, mask-based restatement written with torch ops (every expert is
    evaluated for every token; selection enters through a 0/1 mask)."""
    t = {n: torch.tensor(np.asarray(v, dtype=np.float64), requires_grad=True) for n, v in p.items()
         if v is not None}
    y = torch.tensor(np.asarray(y1, dtype=np.float64), requires_grad=True)
    if norm == "rms":
        n = y * torch.rsqrt((y * y).mean(-1, keepdim=True) + eps) * t["norm_gamma"]
    else:
        n = y
    u = torch.nn.functional.linear(n, t["w_up"])
    L = torch.nn.functional.linear(u, t["w_router"], t.get("b_router"))
    top = torch.topk(L, k, dim=-1)
    mask = torch.zeros_like(L).scatter(1, top.indices, 1.0)
    w = torch.softmax(L.masked_fill(mask == 0, float("-inf")), dim=-1)       # zero off the top-k
    a = torch.einsum("td,eid->tei", u, t["w_gate"])
    b = torch.einsum("td,eid->tei", u, t["w_upx"])
    f = torch.einsum("tei,edi->ted", torch.nn.functional.silu(a) * b, t["w_downx"])
    z = (w[..., None] * f).sum(1)
    if "ws_gate" in t:
        hs = torch.nn.functional.silu(torch.nn.functional.linear(u, t["ws_gate"])) * \
            torch.nn.functional.linear(u, t["ws_up"])
        z = z + torch.sigmoid(u @ t["ws_sgate"])[:, None] * torch.nn.functional.linear(hs, t["ws_down"])
    return torch.nn.functional.linear(z, t["w_down"]), y, t


@pytest.mark.parametrize("seed,shared,bias", [(0, True, False), (1, False, True), (2, True, True)])
def test_forward_and_backward_match_torch_autograd(seed, shared, bias):
    cfg, p, s = _tiny(seed, d_shared=10 if shared else 0)
    if bias:
        p["b_router"] = np.linspace(-0.3, 0.3, cfg.n_experts).astype(np.float32)
    F_t, y, t = _torch_branch(p, s["y1"], cfg.top_k)
    F, info = orc.branch(p, s["y1"], cfg.top_k)
    assert info["margin"].min() > 1e-6
    assert np.allclose(F, F_t.detach().numpy(), rtol=1e-11, atol=1e-13)
    G = torch.tensor(s["dy2"].astype(np.float64))
    (F_t * G).sum().backward()
    out = orc.backward(p, s["y1"], s["dy2"], cfg.top_k)
    assert np.allclose(out["dy1"], y.grad.numpy(), rtol=1e-9, atol=1e-12)
    for name, tt in t.items():
        ref = tt.grad.numpy() if tt.grad is not None else np.zeros(tt.shape)
        assert np.allclose(out[name], ref, rtol=1e-9, atol=1e-12), name
        if name not in ("b_router",):
            assert np.abs(ref).max() > 0, name       # the comparison is not vacuous


# ------------------------------------------------------------------ finite differences
def _loss(p, y1, G, cfg, route):
    F, _ = orc.branch(p, y1, cfg.top_k, route_override=route)
    return float(np.sum(F * G))


@pytest.mark.parametrize("seed", [0, 4])
def test_backward_matches_central_differences(seed):
    cfg, p, s = _tiny(seed)
    p["b_router"] = np.linspace(0.2, -0.2, cfg.n_experts).astype(np.float32)
    p = {n: np.asarray(v, dtype=np.float64) for n, v in p.items()}
    y1 = s["y1"].astype(np.float64)
    G = s["dy2"].astype(np.float64)
    _, info = orc.branch(p, y1, cfg.top_k)
    assert info["margin"].min() > 1e-3, "pick a seed with clear routing margins"
    out = orc.backward(p, y1, G, cfg.top_k)
    rng = np.random.default_rng(seed)
    step = 1e-6

    def fd(tensor_name, index):
        def at(delta):
            q = dict(p)
            yy = y1
            if tensor_name == "y1":
                yy = y1.copy(); yy[index] += delta
            else:
                a = p[tensor_name].copy(); a[index] += delta; q[tensor_name] = a
            return _loss(q, yy, G, cfg, None)
        return (at(step) - at(-step)) / (2 * step)

    names = ["y1"] + [n for n in p]
    for name in names:
        arr = y1 if name == "y1" else p[name]
        grad = out["dy1"] if name == "y1" else out[name]
        assert grad.shape == arr.shape, name
        for _ in range(6):
            index = tuple(int(rng.integers(0, n)) for n in arr.shape)
            num = fd(name, index)
            assert grad[index] == pytest.approx(num, rel=2e-6, abs=2e-9), (name, index)
        # one directional derivative over the whole tensor
        v = rng.standard_normal(arr.shape)

        def at(delta):
            q = dict(p); yy = y1
            if name == "y1":
                yy = y1 + delta * v
            else:
                q[name] = p[name] + delta * v
            return _loss(q, yy, G, cfg, None)
        num = (at(step) - at(-step)) / (2 * step)
        assert float(np.sum(grad * v)) == pytest.approx(num, rel=2e-6, abs=2e-9), name


def test_backward_linear_in_upstream_gradient():
    cfg, p, s = _tiny(5)
    G = s["dy2"].astype(np.float64)
    a = orc.backward(p, s["y1"], G, cfg.top_k)
    b = orc.backward(p, s["y1"], -2.5 * G, cfg.top_k)
    for name in ("dy1", "w_up", "w_gate", "w_router", "ws_sgate", "norm_gamma"):
        assert np.allclose(b[name], -2.5 * a[name], rtol=1e-12, atol=1e-15), name
    assert np.array_equal(a["dx2"], s["dy2"].astype(np.float64))       # dX2 = dY2 exactly


# ------------------------------------------------------------------ special cases
def test_single_expert_is_dense_swiglu_mlp():
    cfg, p, s = _tiny(6, n_experts=1, top_k=1, d_shared=0)
    F, info = orc.branch(p, s["y1"], 1, norm="none")
    assert np.allclose(info["gates"], 1.0)
    y = s["y1"].astype(np.float64)
    u = y @ p["w_up"].astype(np.float64).T
    a = u @ p["w_gate"][0].astype(np.float64).T
    b = u @ p["w_upx"][0].astype(np.float64).T
    ref = ((a / (1 + np.exp(-a))) * b) @ p["w_downx"][0].astype(np.float64).T @ p["w_down"].astype(np.float64).T
    assert np.allclose(F, ref, rtol=1e-12, atol=1e-14)


def test_k_equals_E_is_full_softmax_mixture():
    cfg, p, s = _tiny(7, d_shared=0)
    E = cfg.n_experts
    F, info = orc.branch(p, s["y1"], E)
    L = info["logits"]
    w = np.exp(L - L.max(1, keepdims=True)); w /= w.sum(1, keepdims=True)
    u = orc.norm_fwd(s["y1"], p["norm_gamma"], 1e-6)[0] @ p["w_up"].astype(np.float64).T
    z = np.zeros_like(u)
    for e in range(E):
        a = u @ p["w_gate"][e].astype(np.float64).T
        b = u @ p["w_upx"][e].astype(np.float64).T
        z += w[:, e:e + 1] * ((a / (1 + np.exp(-a)) * b) @ p["w_downx"][e].astype(np.float64).T)
    assert np.allclose(F, z @ p["w_down"].astype(np.float64).T, rtol=1e-12, atol=1e-14)


def test_identical_experts_make_routing_irrelevant():
    cfg, p, s = _tiny(8, d_shared=0)
    for n in ("w_gate", "w_upx", "w_downx"):
        p[n] = np.repeat(p[n][:1], cfg.n_experts, axis=0)
    F, _ = orc.branch(p, s["y1"], cfg.top_k)
    F_other, _ = orc.branch(p, s["y1"], cfg.top_k,
                            route_override=np.tile(np.array([3, 4]), (cfg.tokens, 1)))
    # gate weights sum to one, so any selection gives f(u); compare with a 1-expert block
    q = dict(p); q["w_router"] = p["w_router"][:1]
    for n in ("w_gate", "w_upx", "w_downx"):
        q[n] = p[n][:1]
    F1, _ = orc.branch(q, s["y1"], 1)
    assert np.allclose(F, F1, rtol=1e-12, atol=1e-14)
    assert np.allclose(F_other, F1, rtol=1e-12, atol=1e-14)


def test_zero_down_adapter_is_identity_coupling():
    cfg, p, s = _tiny(9)
    p["w_down"] = np.zeros_like(p["w_down"])
    y2, _ = orc.forward(p, s["y1"], s["x2"], cfg.top_k)
    assert np.array_equal(y2, s["x2"].astype(np.float64))
    out = orc.backward(p, s["y1"], s["dy2"], cfg.top_k)
    assert np.abs(out["dy1"]).max() == 0.0
    assert np.abs(out["w_down"]).max() > 0.0


def test_token_permutation_equivariance():
    cfg, p, s = _tiny(10)
    perm = np.random.default_rng(0).permutation(cfg.tokens)
    F, _ = orc.branch(p, s["y1"], cfg.top_k)
    Fp, _ = orc.branch(p, s["y1"][perm], cfg.top_k)
    assert np.allclose(Fp, F[perm], rtol=1e-13, atol=1e-15)
    a = orc.backward(p, s["y1"], s["dy2"], cfg.top_k)
    b = orc.backward(p, s["y1"][perm], s["dy2"][perm], cfg.top_k)
    assert np.allclose(b["dy1"], a["dy1"][perm], rtol=1e-12, atol=1e-15)
    for name in ("w_up", "w_down", "w_gate", "w_upx", "w_downx", "w_router", "ws_gate", "norm_gamma"):
        assert np.allclose(a[name], b[name], rtol=1e-10, atol=1e-14), name


def test_rmsnorm_scale_invariance():
    cfg, p, s = _tiny(11)
    y = s["y1"].astype(np.float64)
    F, _ = orc.branch(p, y, cfg.top_k, eps=0.0)
    Fc, _ = orc.branch(p, 37.5 * y, cfg.top_k, eps=0.0)
    assert np.allclose(F, Fc, rtol=1e-11, atol=1e-13)
    n, r = orc.norm_fwd(s["y1"], None, 0.0)
    assert np.allclose(np.mean(n * n, axis=1), 1.0, atol=1e-13)


def test_suppressed_expert_is_never_selected_and_gets_no_gradient():
    cfg, p, s = _tiny(12)
    b = np.zeros(cfg.n_experts, dtype=np.float32); b[2] = -1e4
    p["b_router"] = b
    out = orc.backward(p, s["y1"], s["dy2"], cfg.top_k)
    assert not (out["idx"] == 2).any()
    for name in ("w_gate", "w_upx", "w_downx"):
        assert np.abs(out[name][2]).max() == 0.0
    assert np.abs(out["w_router"][2]).max() == 0.0 and out["b_router"][2] == 0.0
    assert np.abs(out["w_gate"]).max() > 0.0


def test_route_override_changes_only_selection():
    cfg, p, s = _tiny(13)
    _, info = orc.branch(p, s["y1"], cfg.top_k)
    F2, info2 = orc.branch(p, s["y1"], cfg.top_k, route_override=info["idx"])
    F1, _ = orc.branch(p, s["y1"], cfg.top_k)
    assert np.array_equal(F1, F2)


# ------------------------------------------------------------------ library cross-check of MLP_pt
@pytest.mark.parametrize("gating,norm_topk", [("renorm", True), ("softmax_all", False)])
def test_mlp_pt_matches_transformers_qwen2_moe_block(gating, norm_topk):
    m = pytest.importorskip("transformers.models.qwen2_moe.modeling_qwen2_moe")
    cfg, p, s = _tiny(14, d_model=32, n_experts=6, top_k=3, d_expert=16, d_shared=24)
    try:
        hf_cfg = m.Qwen2MoeConfig(hidden_size=cfg.d_model, moe_intermediate_size=cfg.d_expert,
                                  shared_expert_intermediate_size=cfg.d_shared,
                                  num_experts=cfg.n_experts, num_experts_per_tok=cfg.top_k,
                                  norm_topk_prob=norm_topk)
        blk = m.Qwen2MoeSparseMoeBlock(hf_cfg).double()
        sd = blk.state_dict()
        T = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
        new = {
            "gate.weight": T(p["w_router"]),
            "experts.gate_up_proj": T(np.concatenate([p["w_gate"], p["w_upx"]], axis=1)),
            "experts.down_proj": T(p["w_downx"]),
            "shared_expert.gate_proj.weight": T(p["ws_gate"]),
            "shared_expert.up_proj.weight": T(p["ws_up"]),
            "shared_expert.down_proj.weight": T(p["ws_down"]),
            "shared_expert_gate.weight": T(p["ws_sgate"])[None, :],
        }
        if set(new) != set(sd) or any(new[k].shape != sd[k].shape for k in new):
            pytest.skip("installed transformers lays the block out differently")
        blk.load_state_dict(new)
    except (TypeError, AttributeError) as exc:      # API drift in the library
        pytest.skip(f"transformers API differs: {exc}")
    # feed MLP_pt directly: identity adapters on a d-wide input, no norm
    q = dict(p)
    q["w_up"] = np.eye(cfg.d_model); q["w_down"] = np.eye(cfg.d_model); q["norm_gamma"] = None
    u = np.random.default_rng(3).standard_normal((9, cfg.d_model))
    F, info = orc.branch(q, u, cfg.top_k, norm="none", gating=gating)
    with torch.no_grad():
        ref = blk(torch.tensor(u)[None])
    ref = ref[0] if isinstance(ref, tuple) else ref
    # the library evaluates its gate softmax in fp32, hence the tolerance; a swapped
    # operand or a different normalisation is off by orders of magnitude more
    assert np.allclose(F, ref.reshape(9, cfg.d_model).numpy(), rtol=1e-6, atol=1e-7)


# ------------------------------------------------------------------ gating without renormalisation
def test_softmax_all_gates_are_the_renormalised_gates_times_the_selected_mass():
    cfg, p, s = _tiny(21)
    _, a = orc.forward(p, s["y1"], s["x2"], cfg.top_k, gating="softmax_all")
    _, r = orc.forward(p, s["y1"], s["x2"], cfg.top_k, gating="renorm")
    assert np.array_equal(a["idx"], r["idx"])                       # the same experts are selected
    L = a["logits"]
    prob = np.exp(L) / np.exp(L).sum(axis=1, keepdims=True)         # textbook softmax over all experts
    mass = np.take_along_axis(prob, a["idx"], axis=1).sum(axis=1)
    assert (mass < 1).all() and (mass > 0).all()
    assert np.allclose(a["gates"].sum(axis=1), mass, rtol=1e-13)
    assert np.allclose(a["gates"], r["gates"] * mass[:, None], rtol=1e-13)
    assert np.allclose(a["gates"], np.take_along_axis(prob, a["idx"], axis=1), rtol=1e-13)


def test_softmax_all_equals_renorm_when_every_expert_is_selected():
    cfg, p, s = _tiny(22, top_k=5)
    Fa, _ = orc.branch(p, s["y1"], cfg.top_k, gating="softmax_all")
    Fr, _ = orc.branch(p, s["y1"], cfg.top_k, gating="renorm")
    assert np.allclose(Fa, Fr, rtol=1e-12, atol=1e-14)
    ga = orc.backward(p, s["y1"], s["dy2"], cfg.top_k, gating="softmax_all")
    gr = orc.backward(p, s["y1"], s["dy2"], cfg.top_k, gating="renorm")
    for n in ("dy1", "w_router", "w_gate", "w_up", "ws_sgate"):
        assert np.allclose(ga[n], gr[n], rtol=1e-10, atol=1e-13), n


@pytest.mark.parametrize("seed", [23, 24])
def test_softmax_all_backward_matches_central_differences(seed):
    """Here the unselected logits carry gradient too (through the softmax denominator)."""
    cfg, p, s = _tiny(seed)
    for n in p:
        p[n] = p[n].astype(np.float64)
    y1, dy2 = s["y1"].astype(np.float64), s["dy2"].astype(np.float64)
    _, info = orc.branch(p, y1, cfg.top_k, gating="softmax_all")
    assert info["margin"].min() > 1e-3
    g = orc.backward(p, y1, dy2, cfg.top_k, gating="softmax_all")
    loss = lambda: float(np.sum(dy2 * orc.branch(p, y1, cfg.top_k, gating="softmax_all")[0]))
    rng = np.random.default_rng(seed)
    eps = 1e-6
    for _ in range(6):
        t, i = int(rng.integers(cfg.tokens)), int(rng.integers(cfg.h))
        old = y1[t, i]
        y1[t, i] = old + eps; lp = loss()
        y1[t, i] = old - eps; lm = loss()
        y1[t, i] = old
        fd = (lp - lm) / (2 * eps)
        assert abs(fd - g["dy1"][t, i]) <= 1e-6 * max(1.0, abs(fd)), (t, i, fd, g["dy1"][t, i])
    for name in ("w_router", "w_up", "w_downx", "ws_gate"):
        W = p[name]
        for _ in range(3):
            pos = tuple(int(rng.integers(n)) for n in W.shape)
            old = W[pos]
            W[pos] = old + eps; lp = loss()
            W[pos] = old - eps; lm = loss()
            W[pos] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - g[name][pos]) <= 2e-6 * max(1.0, abs(fd)), (name, pos, fd, g[name][pos])
    # the router gradient is dense now: experts that were never selected still get one
    never = np.setdiff1d(np.arange(cfg.n_experts), np.unique(info["idx"]))
    if never.size:
        assert np.abs(g["w_router"][never]).max() > 0


# ------------------------------------------------------------------ optimiser step
def test_sgd_step_descends_by_lr_times_the_squared_gradient_norm():
    """Pins sign and scale of the update against the forward map alone: for L(W) = <dY2, Y2(W)> a step
    W' = W - lr * g changes L by -lr * |g|^2 to first order, so (L(W') - L(W)) / lr -> -|g|^2 as lr -> 0,
    with an error that shrinks in proportion to lr.  Only the named weights may move."""
    cfg, p, s = _tiny(seed=4, top_k=5)          # k = E: smooth everywhere, no routing jumps
    G = np.random.default_rng(2).standard_normal(s["x2"].shape)

    def loss(q):
        y2, _ = orc.forward(q, s["y1"], s["x2"], cfg.top_k, cfg.norm_eps)
        return float(np.sum(G * y2))

    g = orc.backward(p, s["y1"], G, cfg.top_k, cfg.norm_eps)
    names = ("w_up", "w_gate", "w_downx", "ws_up")
    sq = sum(float(np.sum(g[n] ** 2)) for n in names)
    L0 = loss(p)
    errs = []
    for lr in (1e-4, 1e-5):
        q = orc.sgd_step(p, g, lr, names)
        for n in p:
            if n in names:
                assert np.allclose(q[n], np.asarray(p[n], np.float64) - lr * g[n], rtol=0, atol=0)
            else:
                assert q[n] is p[n]
        errs.append(abs((loss(q) - L0) / lr + sq) / sq)
    assert errs[0] < 2e-2 and errs[1] < errs[0] / 5          # first-order term exact, remainder O(lr)
    # an ascent step does the opposite
    up = orc.sgd_step(p, g, -1e-5, names)
    assert loss(up) > L0 > loss(orc.sgd_step(p, g, 1e-5, names))


# ------------------------------------------------------------------ FP8 variant of the routed experts
def _e4m3_table():
    """Every finite e4m3 value from the format's definition: 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits,
    exponent field 0 = subnormal, the code S.1111.111 is NaN, no infinities."""
    vals = []
    for ebits in range(16):
        for m in range(8):
            if ebits == 15 and m == 7:
                continue
            vals.append(m / 8 * 2.0 ** -6 if ebits == 0 else (1 + m / 8) * 2.0 ** (ebits - 7))
    return np.array(sorted(set(vals)))


def test_e4m3_rounding_against_the_value_table_and_the_library_cast():
    tab = _e4m3_table()
    assert tab.max() == 448.0 and tab[1] == 2.0 ** -9 and len(tab) == 127
    assert np.array_equal(orc.e4m3_round(tab.astype(np.float32)), tab.astype(np.float32))          # representable values stay
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 100, rng.standard_normal(20000) * 0.01, rng.uniform(-448, 448, 20000),
                        (tab[:-1] + tab[1:]) / 2, -(tab[:-1] + tab[1:]) / 2]).astype(np.float32)      # incl. every tie
    got = orc.e4m3_round(x)
    # brute force: nearest table value, ties to the even mantissa (= even position in the table), saturation
    a = np.minimum(np.abs(x.astype(np.float64)), 448.0)
    j = np.searchsorted(tab, a)
    lo, hi = tab[np.maximum(j - 1, 0)], tab[np.minimum(j, len(tab) - 1)]
    pick_hi = (hi - a < a - lo) | ((hi - a == a - lo) & (np.minimum(j, len(tab) - 1) % 2 == 0))
    want = np.sign(x) * np.where(pick_hi, hi, lo)
    assert np.array_equal(got.astype(np.float64), want)
    # the installed library's cast (no saturation there: stay inside the finite range)
    inside = np.abs(x) <= 448
    lib = torch.from_numpy(x[inside]).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(got[inside], lib)
    assert np.array_equal(orc.e4m3_round(np.array([449, 1e6, -500], np.float32)), np.array([448, 448, -448], np.float32))
    # bf16 rounding against the library's cast
    y = (rng.standard_normal(50000) * 3).astype(np.float32)
    assert np.array_equal(orc.round_bf16(y), torch.from_numpy(y).to(torch.bfloat16).to(torch.float32).numpy())


def test_row_quantisation_scales_and_error_bound():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((37, 96)) * rng.uniform(0.01, 30, (37, 1))).astype(np.float32)
    x[5] = 0
    q, s = orc.quantize_rows_e4m3(x)
    assert s[5] == 1 and (q[5] == 0).all()
    assert np.allclose(np.abs(q).max(axis=1)[np.arange(37) != 5], 448.0)          # the row maximum maps onto the largest code
    back = q * s[:, None]
    # relative error of a normal e4m3 value is at most 2^-4; tiny entries sit on the subnormal grid 2^-9 * scale
    assert (np.abs(back - x) <= np.maximum(np.abs(x) * 2.0 ** -4, s[:, None] * 2.0 ** -10) * (1 + 1e-6)).all()
    # a product of quantised operands is the product of the dequantised ones
    w = (rng.standard_normal((11, 96)) * 0.05).astype(np.float32)
    wq, ws_ = orc.quantize_rows_e4m3(w)
    f64 = np.float64
    assert np.allclose(orc.fp8_matmul(q, s, wq, ws_), (q.astype(f64) * s.astype(f64)[:, None]) @ (wq.astype(f64) * ws_.astype(f64)[:, None]).T, rtol=1e-12)


def test_fp8_experts_is_the_branch_with_quantised_expert_operands():
    """Written a second time with the library's casts: the FP8 branch equals the plain branch evaluated on
    dequantised operands at the three expert products; and it stays within the format's error of the exact one."""
    cfg, p, s = _tiny(seed=6, d_model=64, d_expert=32, d_shared=32, tokens=19)
    F8, info = orc.branch(p, s["y1"], cfg.top_k, cfg.norm_eps, fp8_experts=True)
    F, info0 = orc.branch(p, s["y1"], cfg.top_k, cfg.norm_eps)
    assert np.array_equal(info["idx"], info0["idx"]) and np.allclose(info["gates"], info0["gates"])     # routing is untouched

    def q8(t):      # per-row e4m3 through torch, dequantised
        amax = t.abs().amax(dim=-1, keepdim=True)
        sc = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
        return (t * (1.0 / sc)).to(torch.float8_e4m3fn).to(torch.float32).double() * sc.double()

    n, _ = orc.norm_fwd(s["y1"], p["norm_gamma"], cfg.norm_eps)
    u = n @ p["w_up"].astype(np.float64).T
    z = np.zeros_like(u)
    for t in range(cfg.tokens):
        ub = q8(torch.from_numpy(u[t:t + 1].astype(np.float32)).to(torch.bfloat16).float())
        for slot, e in enumerate(info["idx"][t]):
            a = ub @ q8(torch.from_numpy(p["w_gate"][e])).T
            b = ub @ q8(torch.from_numpy(p["w_upx"][e])).T
            hg = (info["gates"][t, slot] * torch.nn.functional.silu(a) * b).float().to(torch.bfloat16).float()
            z[t] += (q8(hg) @ q8(torch.from_numpy(p["w_downx"][e])).T).numpy()[0]
    a_s = u @ p["ws_gate"].astype(np.float64).T
    S = (orc.silu(a_s) * (u @ p["ws_up"].astype(np.float64).T)) @ p["ws_down"].astype(np.float64).T
    z += info["sgate"][:, None] * S
    assert np.allclose(F8, z @ p["w_down"].astype(np.float64).T, rtol=1e-9, atol=1e-12)
    err = np.linalg.norm(F8 - F) / np.linalg.norm(F)
    assert 1e-3 < err < 1e-1          # the quantisation is visible, and of the size three bits of mantissa give
    # forward then inverse with the same arithmetic reconstructs exactly
    y2, _ = orc.forward(p, s["y1"], s["x2"], cfg.top_k, cfg.norm_eps, fp8_experts=True)
    x2, _ = orc.inverse(p, s["y1"], y2, cfg.top_k, cfg.norm_eps, fp8_experts=True)
    assert np.max(np.abs(x2 - s["x2"])) < 1e-10


def test_adam_step_is_the_library_optimiser():
    """adam_step against torch.optim.Adam / AdamW (an independent implementation of the same rule) over three
    steps with changing gradients, and its first step in closed form: from zero moments the step is
    -lr * g / (|g| + eps), whatever beta1 and beta2 are."""
    rng = np.random.default_rng(11)
    w0 = {"a": rng.standard_normal((5, 7)), "b": rng.standard_normal((3,))}
    gs = [{n: rng.standard_normal(v.shape) * 10.0 ** rng.integers(-3, 2) for n, v in w0.items()} for _ in range(3)]
    for wd in (0.0, 0.1):
        tw = {n: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for n, v in w0.items()}
        opt = (torch.optim.AdamW if wd else torch.optim.Adam)(list(tw.values()), lr=3e-3, betas=(0.8, 0.95), eps=1e-6,
                                                              **({"weight_decay": wd} if wd else {}))
        w, m, v = dict(w0), {}, {}
        for t, g in enumerate(gs, start=1):
            for n in tw:
                tw[n].grad = torch.tensor(g[n], dtype=torch.float64)
            opt.step()
            w, m, v = orc.adam_step(w, g, m, v, 3e-3, t, list(w0), beta1=0.8, beta2=0.95, eps=1e-6, weight_decay=wd)
            for n in w0:
                assert np.allclose(w[n], tw[n].detach().numpy(), rtol=1e-12, atol=1e-14), (n, t, wd)
    w1, m1, v1 = orc.adam_step(w0, gs[0], {}, {}, 1e-2, 1, ["a"], beta1=0.3, beta2=0.7, eps=1e-9)
    g = gs[0]["a"]
    assert np.allclose(w1["a"] - w0["a"], -1e-2 * g / (np.abs(g) + 1e-9), rtol=1e-9)
    assert np.allclose(m1["a"], 0.7 * g) and np.allclose(v1["a"], 0.3 * g * g) and w1["b"] is w0["b"]
