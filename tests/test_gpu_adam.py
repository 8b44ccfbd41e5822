"""Adam fused into the weight-gradient products (revffn_moe_backward_adam) against the oracle's gradients
followed by the oracle's adam_step.

What is compared, and at which tolerance.  The kernels' gradient g differs from the oracle's by the gradient
tolerance (relative L2 2e-2 for bf16 products, 1e-4 for fp32), so
  * the first moment, through (m_new - beta1 m_old) / (1 - beta1) = g, is held to that tolerance;
  * the second moment, through (v_new - beta2 v_old) / (1 - beta2) = g^2, to twice it (a square doubles a
    relative error);
  * the step W_new - W_old (read from the fp32 master copy, so that bf16 rounding of the stored weight does not
    enter) to twice it as well: it is lr m^ / (sqrt(v^) + eps), a ratio of the two.
The stored bf16 weight must be the rounded master value bit for bit, and everything not in the mask (stream
gradient, remaining gradients) must equal the plain pass bit for bit.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, grad_buffers, make_block, rel_l2, to_device_weights

pytestmark = pytest.mark.gpu

TOL_BF16, TOL_F32 = 2e-2, 1e-4
B1, B2, EPS, WD, STEP = 0.8, 0.9, 1e-6, 0.05, 3


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def _weights(cfg, seed, scale=4.0):
    w = make_weights(cfg, seed)
    for n in w:
        if n not in ("norm_gamma", "b_router"):
            w[n] = w[n] * scale
            if cfg.weight_dtype == "bf16":
                w[n] = to_bf16_values(w[n])
    return w


def _moments(ref, names, seed):
    """Moment estimates of the size earlier steps would have left: m ~ g-sized noise, v ~ g^2-sized, positive."""
    rng = np.random.default_rng(seed)
    mom, var = {}, {}
    for n in names:
        rms = float(np.sqrt(np.mean(ref[n] ** 2))) + 1e-30
        mom[n] = (rng.standard_normal(ref[n].shape) * rms).astype(np.float32)
        var[n] = ((rng.standard_normal(ref[n].shape) * rms) ** 2 + 0.1 * rms * rms).astype(np.float32)
    return mom, var


def _run(rv, cfg, w, s, names, tol, flags=0, lr=None):
    blk = make_block(cfg, w, flags=flags)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    blk.forward(y1, x2, topk_idx_out=idx)
    ref = orc.backward(w, s["y1"], s["dy2"], cfg.top_k, cfg.norm_eps, route_override=idx.cpu().numpy())
    dy1_p, g_p = torch.zeros_like(y1), grad_buffers(cfg, w)
    blk.backward(y1, dy2, dy1_p, g_p, topk_idx_in=idx)                       # the plain pass, for what must not change
    mom0, var0 = _moments(ref, names, 5)
    mom = {n: dev(mom0[n]) for n in names}
    var = {n: dev(var0[n]) for n in names}
    masters = {n: blk.weights[n].float().clone() for n in names}
    w_old = {n: masters[n].cpu().numpy().astype(np.float64) for n in names}
    lr = lr if lr is not None else 0.05 * float(np.sqrt(np.mean(w[names[0]] ** 2)))
    rest = {n: t for n, t in grad_buffers(cfg, w).items() if n not in names}
    dy1 = torch.zeros_like(y1)
    adam = rv.make_adam(lr, STEP, names, mom, var, masters, beta1=B1, beta2=B2, eps=EPS, weight_decay=WD)
    blk.backward(y1, dy2, dy1, rest, topk_idx_in=idx, sgd=adam)
    assert blk.status() == 0
    assert torch.equal(dy1, dy1_p)
    for n, t in rest.items():
        assert torch.equal(t, g_p[n]), n
    new, m_ref, v_ref = orc.adam_step(w, ref, mom0, var0, lr, STEP, names, beta1=B1, beta2=B2, eps=EPS, weight_decay=WD)
    for n in names:
        m_new, v_new = mom[n].cpu().numpy().astype(np.float64), var[n].cpu().numpy().astype(np.float64)
        g_from_m = (m_new - B1 * mom0[n]) / (1 - B1)
        g2_from_v = (v_new - B2 * var0[n]) / (1 - B2)
        assert rel_l2(g_from_m, ref[n]) <= tol, (n, rel_l2(g_from_m, ref[n]))
        assert rel_l2(g2_from_v, ref[n] ** 2) <= 2 * tol, (n, rel_l2(g2_from_v, ref[n] ** 2))
        assert rel_l2(m_new, m_ref[n]) <= tol and rel_l2(v_new, v_ref[n]) <= 2 * tol, n
        step = masters[n].cpu().numpy().astype(np.float64) - w_old[n]
        assert rel_l2(step, new[n] - w[n]) <= 2 * tol, (n, rel_l2(step, new[n] - w[n]))
        if cfg.weight_dtype == "bf16":
            assert torch.equal(blk.weights[n], masters[n].to(torch.bfloat16)), n
        else:
            assert torch.equal(blk.weights[n], masters[n]), n
    return blk


@pytest.mark.parametrize("simt", [True, False])
def test_fused_adam_matches_oracle_gradients_and_step(rv, simt):
    cfg = BlockConfig("U", tokens=333, d_model=256, n_experts=8, top_k=3, d_expert=128, d_shared=256, weight_dtype="bf16")
    w, s = _weights(cfg, 31), make_streams(cfg, 31)
    _run(rv, cfg, w, s, list(rv.UPD_NAMES), TOL_BF16, flags=rv.FLAG_FORCE_SIMT if simt else 0)


def test_fused_adam_on_the_second_stream_and_a_partial_mask(rv):
    """A larger batch (the weight-gradient products run on the library's second stream, as in every tensor-core
    case); only the experts and one adapter are in the mask, the other gradients are written as usual."""
    cfg = BlockConfig("U", tokens=1300, d_model=256, n_experts=5, top_k=2, d_expert=128, d_shared=256, weight_dtype="bf16")
    w, s = _weights(cfg, 32), make_streams(cfg, 32)
    _run(rv, cfg, w, s, ["w_up", "w_gate", "w_upx", "w_downx"], TOL_BF16)


def test_fused_adam_fp32_block(rv):
    cfg = CONFIGS["C0"]
    w, s = _weights(cfg, 33, 5.0), make_streams(cfg, 33)
    _run(rv, cfg, w, s, ["w_up", "w_down", "w_gate", "w_upx", "w_downx"], TOL_F32)


def test_fused_adam_argument_checks(rv):
    cfg = BlockConfig("U", tokens=64, d_model=256, n_experts=4, top_k=2, d_expert=128, d_shared=0, weight_dtype="bf16")
    w, s = _weights(cfg, 34), make_streams(cfg, 34)
    blk = make_block(cfg, w)
    y1, dy2 = dev(s["y1"]), dev(s["dy2"])
    m = {"w_up": torch.zeros(cfg.d_model, cfg.h, device="cuda")}
    v = {"w_up": torch.zeros(cfg.d_model, cfg.h, device="cuda")}
    before = blk.weights["w_up"].clone()
    with pytest.raises(rv.RevffnError) as e:                                  # the step counter starts at 1
        blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=rv.make_adam(1e-3, 0, ["w_up"], m, v))
    assert e.value.code == -2
    with pytest.raises(rv.RevffnError) as e:                                  # a matrix in the mask without moments
        blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=rv.make_adam(1e-3, 1, ["w_up", "w_down"], m, v))
    assert e.value.code == -1
    assert torch.equal(blk.weights["w_up"], before)                           # refused calls launched nothing
    # first step from zero moments: every element moves by lr * g / (|g| + eps), i.e. by about lr
    master = {"w_up": before.float().clone()}
    blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=rv.make_adam(1e-2, 1, ["w_up"], m, v, master, eps=1e-12))
    assert blk.status() == 0
    moved = (master["w_up"] - before.float()).abs()
    g_nonzero = m["w_up"].abs() > 1e-6
    assert g_nonzero.float().mean() > 0.9
    assert torch.allclose(moved[g_nonzero], torch.full_like(moved[g_nonzero], 1e-2), rtol=1e-3)


def test_reversible_stack_sweep_as_one_adam_step(rv):
    """Three layers: forward, then the reversible sweep with the fused Adam update per layer.  Every layer's
    master weights must move as the oracle's adam_step moves them on the gradients of the oracle's reversible
    back-propagation, and the rebuilt inputs and input gradients must be those of the sweep without updates."""
    cfg = BlockConfig("U", tokens=210, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=256, weight_dtype="bf16")
    L = 3
    ws_host = [_weights(cfg, 40 + l) for l in range(L)]
    weights = [to_device_weights(cfg, w) for w in ws_host]
    stk = rv.Stack(weights=weights, tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k,
                   d_expert=cfg.d_expert, d_shared=cfg.d_shared, weight_dtype=rv.BF16)
    s = make_streams(cfg, 6)
    a, b = dev(s["y1"]), dev(s["x2"])
    idx = torch.empty(L, cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    stk.forward(a, b, idx)
    a_out, b_out = a.clone(), b.clone()
    g0 = dev(s["dy2"])
    ga, gb = g0.clone(), g0.clone()
    stk.backward(a, b, ga, gb, stk.grads_array([{}] * L), topk_idx=idx)                 # the sweep without updates
    _, _, _, _, grads = orc.stack_backward(ws_host, a_out.cpu().numpy(), b_out.cpu().numpy(), s["dy2"], s["dy2"],
                                           cfg.top_k, cfg.norm_eps, route_overrides=idx.cpu().numpy())
    names = list(rv.UPD_NAMES)
    lr = 0.05 * float(np.sqrt(np.mean(ws_host[0]["w_up"] ** 2)))
    structs, state = [], []
    for l in range(L):
        mom0, var0 = _moments(grads[l], names, 50 + l)
        mom = {n: dev(mom0[n]) for n in names}
        var = {n: dev(var0[n]) for n in names}
        masters = {n: weights[l][n].float().clone() for n in names}
        w_old = {n: masters[n].cpu().numpy().astype(np.float64) for n in names}
        structs.append(rv.make_adam(lr, STEP, names, mom, var, masters, beta1=B1, beta2=B2, eps=EPS, weight_decay=WD))
        state.append((mom0, var0, mom, var, masters, w_old))
    a2, b2, ga2, gb2 = a_out.clone(), b_out.clone(), g0.clone(), g0.clone()
    stk.backward(a2, b2, ga2, gb2, stk.grads_array([{}] * L), topk_idx=idx, sgd=structs)
    assert stk.status() == 0
    assert torch.equal(a2, a) and torch.equal(b2, b) and torch.equal(ga2, ga) and torch.equal(gb2, gb)
    for l in range(L):
        mom0, var0, mom, var, masters, w_old = state[l]
        new, m_ref, v_ref = orc.adam_step(ws_host[l], grads[l], mom0, var0, lr, STEP, names, beta1=B1, beta2=B2, eps=EPS,
                                          weight_decay=WD)
        for n in names:
            assert rel_l2(mom[n].cpu().numpy(), m_ref[n]) <= TOL_BF16, (l, n)
            assert rel_l2(var[n].cpu().numpy(), v_ref[n]) <= 2 * TOL_BF16, (l, n)
            step = masters[n].cpu().numpy().astype(np.float64) - w_old[n]
            assert rel_l2(step, new[n] - ws_host[l][n]) <= 2 * TOL_BF16, (l, n, rel_l2(step, new[n] - ws_host[l][n]))
            assert torch.equal(weights[l][n], masters[n].to(torch.bfloat16)), (l, n)
