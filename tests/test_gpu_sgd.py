"""The optimiser step fused into the weight-gradient products (revffn_moe_backward_sgd) against the oracle's
gradients followed by the oracle's sgd_step, and the one-launch form of the experts' gate | up gradients.

Tolerances: the update (W_new - W) / (-lr) is a gradient and is held to the gradient tolerance (relative L2
2e-2 for bf16 products, 1e-4 for the fp32 configuration); lr is chosen large enough that rounding W_new to
bf16 (half a last bit of W) is small against lr * g.  With an fp32 master copy the stored bf16 weight must be
the rounded master value bit for bit.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, grad_buffers, make_block, max_block_rel_l2, rel_l2, to_device_weights

pytestmark = pytest.mark.gpu

TOL_BF16, TOL_F32 = 2e-2, 1e-4


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def _cfg(**kw):
    base = dict(name="U", tokens=300, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=256, weight_dtype="bf16")
    base.update(kw)
    return BlockConfig(**base)


def _weights(cfg, seed, scale=4.0):
    w = make_weights(cfg, seed)
    for n in w:
        if n not in ("norm_gamma", "b_router"):
            w[n] = w[n] * scale
            if cfg.weight_dtype == "bf16":
                w[n] = to_bf16_values(w[n])
    return w


def _lr_for(w, ref, names, frac=0.5):
    """A learning rate at which every named update is at least `frac` of its weight's rms, so that rounding the
    updated weight to bf16 (relative 2^-9 of the new value) stays well below the step itself."""
    return max(frac * float(np.sqrt(np.mean(w[n] ** 2))) / float(np.sqrt(np.mean(ref[n] ** 2))) for n in names)


@pytest.mark.parametrize("simt", [True, False])
@pytest.mark.parametrize("master", [False, True])
def test_fused_sgd_matches_oracle_gradients_and_step(rv, simt, master):
    cfg = _cfg(tokens=333, n_experts=8, top_k=3)
    w, s = _weights(cfg, 21), make_streams(cfg, 21)
    blk = make_block(cfg, w, flags=rv.FLAG_FORCE_SIMT if simt else 0)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    blk.forward(y1, x2, topk_idx_out=idx)
    ref = orc.backward(w, s["y1"], s["dy2"], cfg.top_k, cfg.norm_eps, route_override=idx.cpu().numpy())
    # plain backward first: the gradients the fused form must not change
    dy1_p, g_p = torch.zeros_like(y1), grad_buffers(cfg, w)
    blk.backward(y1, dy2, dy1_p, g_p, topk_idx_in=idx)
    names = list(rv.UPD_NAMES)
    lr = _lr_for(w, ref, names)
    w0 = {n: blk.weights[n].clone() for n in names}
    masters = {n: blk.weights[n].float().clone() for n in names} if master else None
    rest = {n: t for n, t in grad_buffers(cfg, w).items() if n not in names}
    dy1 = torch.zeros_like(y1)
    blk.backward(y1, dy2, dy1, rest, topk_idx_in=idx, sgd=rv.make_sgd(lr, names, masters))
    assert blk.status() == 0
    assert torch.equal(dy1, dy1_p)                                   # the stream gradient does not see the update
    for n, t in rest.items():
        assert torch.equal(t, g_p[n]), n                             # nor do the gradients that are still written
    new = orc.sgd_step(w, ref, lr, names)
    for n in names:
        got = blk.weights[n].float().cpu().numpy()
        step = (got - w0[n].float().cpu().numpy()) / (-lr)
        assert rel_l2(step, ref[n]) <= TOL_BF16, (n, rel_l2(step, ref[n]))
        assert rel_l2(got, new[n]) <= TOL_BF16, n
        if n in ("w_gate", "w_upx", "w_downx"):
            assert max_block_rel_l2(step, ref[n]) <= TOL_BF16, n     # expert by expert
        if master:
            m = masters[n]
            assert torch.equal(blk.weights[n], m.to(torch.bfloat16)), n          # stored weight = rounded master
            assert rel_l2((m.cpu().numpy() - w0[n].float().cpu().numpy()) / (-lr), ref[n]) <= TOL_BF16, n
            # the master keeps what bf16 would drop: it equals W - lr * (the gradient the plain pass wrote) in fp32
            want = w0[n].float() - lr * g_p[n]
            assert torch.allclose(m, want, rtol=1e-5, atol=1e-6), n


def test_fused_sgd_fp32_block(rv):
    cfg = CONFIGS["C0"]
    w, s = _weights(cfg, 22, 5.0), make_streams(cfg, 22)
    blk = make_block(cfg, w)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    blk.forward(y1, x2, topk_idx_out=idx)
    ref = orc.backward(w, s["y1"], s["dy2"], cfg.top_k, cfg.norm_eps, route_override=idx.cpu().numpy())
    names = ["w_up", "w_down", "w_gate", "w_upx", "w_downx"]          # no shared expert in this configuration
    lr = _lr_for(w, ref, names, 0.1)
    blk.backward(y1, dy2, torch.zeros_like(y1), {}, topk_idx_in=idx, sgd=rv.make_sgd(lr, names))
    assert blk.status() == 0
    new = orc.sgd_step(w, ref, lr, names)
    for n in names:
        got = blk.weights[n].cpu().numpy()
        assert rel_l2((got - w[n]) / (-lr), ref[n]) <= TOL_F32, n
        assert rel_l2(got, new[n]) <= TOL_F32, n
    with pytest.raises(rv.RevffnError):                                # a shared-expert bit without a shared expert
        blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=rv.make_sgd(lr, ["ws_up"]))


def test_stage_masks_and_argument_checks(rv):
    cfg = _cfg()
    w, s = _weights(cfg, 23), make_streams(cfg, 23)
    blk = make_block(cfg, w)
    y1, dy2 = dev(s["y1"]), dev(s["dy2"])
    before = {n: t.clone() for n, t in blk.weights.items()}
    # stage 1 of the schedule: only the adapters move
    sgd = rv.Sgd(lr=1e-2, mask=rv.stage_update_mask(1))
    assert sgd.mask == rv.upd_mask(["w_up", "w_down"])
    blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=sgd)
    assert blk.status() == 0
    for n, t in blk.weights.items():
        assert torch.equal(t, before[n]) == (n not in ("w_up", "w_down")), n
    assert rv.stage_update_mask(2) == rv.UPD_ALL
    # a matrix cannot be updated and have its gradient written in the same call
    with pytest.raises(rv.RevffnError) as e:
        blk.backward(y1, dy2, torch.zeros_like(y1), {"w_up": torch.empty(cfg.d_model, cfg.h, device="cuda")},
                     sgd=rv.make_sgd(1e-2, ["w_up"]))
    assert e.value.code == rv.ERR_UNSUPPORTED
    with pytest.raises(rv.RevffnError):
        blk.backward(y1, dy2, torch.zeros_like(y1), {}, sgd=rv.Sgd(lr=1e-2, mask=1 << 9))


@pytest.mark.parametrize("simt", [True, False])
def test_gate_and_up_gradients_from_one_product_equal_the_two_products(rv, simt):
    """Asking for both expert gradients runs one product with M = 2I and two outputs; asking for one of them runs
    the single product.  Same tiles, same K order: bit-identical results."""
    cfg = _cfg(tokens=700, n_experts=5, top_k=2, d_expert=256)
    w, s = _weights(cfg, 24), make_streams(cfg, 24)
    blk = make_block(cfg, w, flags=rv.FLAG_FORCE_SIMT if simt else 0)
    y1, dy2 = dev(s["y1"]), dev(s["dy2"])
    shp = (cfg.n_experts, cfg.d_expert, cfg.d_model)
    both = {n: torch.full(shp, float("nan"), device="cuda") for n in ("w_gate", "w_upx")}
    blk.backward(y1, dy2, torch.zeros_like(y1), both)
    for n in ("w_gate", "w_upx"):
        one = {n: torch.full(shp, float("nan"), device="cuda")}
        blk.backward(y1, dy2, torch.zeros_like(y1), one)
        assert blk.status() == 0
        assert torch.equal(one[n], both[n]), n
    # accumulate works through the two-output form as well
    blk.backward(y1, dy2, torch.zeros_like(y1), both, accumulate=True)
    one = {"w_gate": torch.full(shp, float("nan"), device="cuda")}
    blk.backward(y1, dy2, torch.zeros_like(y1), one)
    assert torch.allclose(both["w_gate"], 2 * one["w_gate"], rtol=1e-6, atol=1e-7)


def test_reversible_stack_sweep_as_one_sgd_step(rv):
    """Three layers: forward, then the reversible sweep with a fused update per layer.  Every layer's weights
    must move by -lr times the gradients the oracle's reversible back-propagation gives, the input gradients and
    the reconstructed inputs must be what the sweep without updates gives."""
    cfg = _cfg(tokens=210, n_experts=6, top_k=2)
    L = 3
    ws_host = [_weights(cfg, 30 + l) for l in range(L)]
    weights = [to_device_weights(cfg, w) for w in ws_host]
    kw = dict(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k, d_expert=cfg.d_expert,
              d_shared=cfg.d_shared, weight_dtype=rv.BF16)
    stk = rv.Stack(weights=weights, **kw)
    s = make_streams(cfg, 5)
    a, b = dev(s["y1"]), dev(s["x2"])
    idx = torch.empty(L, cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    stk.forward(a, b, idx)
    a_out, b_out = a.clone(), b.clone()
    g0 = dev(s["dy2"])
    # reference sweep without updates
    ga, gb = g0.clone(), g0.clone()
    stk.backward(a, b, ga, gb, stk.grads_array([{}] * L), topk_idx=idx)
    A_in, B_in, gA, gB, grads = orc.stack_backward(ws_host, a_out.cpu().numpy(), b_out.cpu().numpy(), s["dy2"], s["dy2"],
                                                   cfg.top_k, cfg.norm_eps, route_overrides=idx.cpu().numpy())
    names = list(rv.UPD_NAMES)
    lr = max(_lr_for(ws_host[l], grads[l], names) for l in range(L))
    w0 = [{n: weights[l][n].float().cpu().numpy() for n in names} for l in range(L)]
    a2, b2, ga2, gb2 = a_out.clone(), b_out.clone(), g0.clone(), g0.clone()
    stk.backward(a2, b2, ga2, gb2, stk.grads_array([{}] * L), topk_idx=idx, sgd=[rv.make_sgd(lr, names)] * L)
    assert stk.status() == 0
    assert torch.equal(a2, a) and torch.equal(b2, b) and torch.equal(ga2, ga) and torch.equal(gb2, gb)
    for l in range(L):
        for n in names:
            step = (weights[l][n].float().cpu().numpy() - w0[l][n]) / (-lr)
            assert rel_l2(step, grads[l][n]) <= TOL_BF16, (l, n, rel_l2(step, grads[l][n]))
