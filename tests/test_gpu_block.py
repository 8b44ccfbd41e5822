"""Parity of whole RevFFN blocks (Eq. 1 then Eq. 2) and stacks of them between the CUDA library, called
through the C ABI, and the CPU oracle: forward, the inverse pass, and reversible back-propagation, which
rebuilds every layer's inputs from its outputs and takes the gradients there.

The expert sets the GPU selected are handed to the oracle (they are checked against the oracle's own
selection wherever the top-k margin is not a near-tie), so that one flipped near-tie does not turn a
rounding difference into a different function."""
import numpy as np
import pytest
import torch

from oracle import revffn_block_oracle as blk
from workloads import BlockConfig, make_weights, to_bf16_values
from workloads.generate import AttnConfig, make_attn_streams, make_attn_weights

from helpers import dev, rel_l2

pytestmark = pytest.mark.gpu

ATTN_F32 = ("norm_gamma", "b_q", "b_k", "b_v")
MOE_F32 = ("norm_gamma", "b_router")


def _make(acfg: AttnConfig, mcfg: BlockConfig, layers: int, std: float, iters: int = 1, flags: int = 0, moe_scale: float = 6.0):
    import paper_2512_20920_b200 as rv
    wdt = torch.bfloat16 if acfg.weight_dtype == "bf16" else torch.float32
    host, dev_a, dev_m = [], [], []
    for l in range(layers):
        pa = make_attn_weights(acfg, 100 + l, std=std, bias_std=std)
        pm = make_weights(mcfg, 7, block=l)
        for n in pm:                                  # scaled up so that the branch output is O(0.1) at these small widths
            if n not in MOE_F32:
                pm[n] = pm[n] * moe_scale
                if mcfg.weight_dtype == "bf16":
                    pm[n] = to_bf16_values(pm[n])
        host.append((pa, pm))
        dev_a.append({n: torch.from_numpy(v).to("cuda", torch.float32 if n in ATTN_F32 else wdt) for n, v in pa.items()})
        dev_m.append({n: torch.from_numpy(v).to("cuda", torch.float32 if n in MOE_F32 else wdt) for n, v in pm.items()})
    st = rv.RevStack(batch=acfg.batch, seq_len=acfg.seq_len, d_model=acfg.d_model, n_heads=acfg.n_heads,
                     n_kv_heads=acfg.n_kv_heads, n_experts=mcfg.n_experts, top_k=mcfg.top_k, d_expert=mcfg.d_expert,
                     d_shared=mcfg.d_shared, weight_dtype=rv.BF16 if acfg.weight_dtype == "bf16" else rv.F32,
                     attn_weights=dev_a, moe_weights=dev_m, inverse_iters=iters, rope_theta=acfg.rope_theta, flags=flags)
    cfg = dict(seq_len=acfg.seq_len, n_heads=acfg.n_heads, n_kv_heads=acfg.n_kv_heads, top_k=mcfg.top_k,
               eps=acfg.norm_eps, theta=acfg.rope_theta)
    return st, host, cfg, dev_a, dev_m


def _run(acfg, mcfg, layers, std, tol, iters=1, flags=0, moe_scale=6.0):
    st, host, cfg, dev_a, dev_m = _make(acfg, mcfg, layers, std, iters, flags, moe_scale)
    s = make_attn_streams(acfg, 5)
    T, k = acfg.tokens, mcfg.top_k
    X1, X2, G1, G2 = s["x1"], s["x2"], s["dy1"], s["dx2"]
    a, b = dev(X1), dev(X2)
    idx = torch.empty(layers, T, k, dtype=torch.int32, device="cuda")
    st.forward(a, b, idx)
    assert st.status() == 0
    ov = [i for i in idx.cpu().numpy()]
    Y1, Y2, infos = blk.stack_forward(host, X1, X2, cfg, ov)
    # the oracle's own selection agrees wherever it is not a near-tie
    _, _, free = blk.stack_forward(host, X1, X2, cfg)
    from oracle import revffn_oracle as moe
    for l in range(layers):
        margin = moe.topk_margin(infos[l]["logits"], k)
        same = (np.sort(ov[l], 1) == np.sort(moe.topk_indices(infos[l]["logits"], k), 1)).all(1)
        assert (same | (margin < 1e-4)).all(), f"layer {l}: selection differs outside a near-tie"
    assert rel_l2(a.cpu().numpy() - X1, Y1 - X1) < tol and rel_l2(b.cpu().numpy() - X2, Y2 - X2) < tol

    # reversible back-propagation from the oracle's outputs (same starting point on both sides)
    y1, y2 = dev(Y1.astype(np.float32)), dev(Y2.astype(np.float32))
    g1, g2 = dev(G1), dev(G2)
    ga_t = [{n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()} for w in dev_a]
    gm_t = [{n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()} for w in dev_m]
    ga, gm = st.grads_arrays(ga_t, gm_t)
    st.backward(y1, y2, g1, g2, ga, gm, idx)
    assert st.status() == 0
    R1, R2, dX1, dX2, grads = blk.stack_backward(host, Y1.astype(np.float32), Y2.astype(np.float32), G1, G2, cfg,
                                                 n_iter=iters, route_overrides=ov)
    # rebuilt inputs: compare what was subtracted, not the streams themselves
    assert rel_l2(Y1 - y1.cpu().numpy(), Y1 - R1) < tol and rel_l2(Y2 - y2.cpu().numpy(), Y2 - R2) < tol
    assert rel_l2(g1.cpu().numpy(), dX1) < tol and rel_l2(g2.cpu().numpy(), dX2) < tol
    for l in range(layers):
        for n in host[l][0]:
            assert rel_l2(ga_t[l][n].cpu().numpy(), grads[l][0][n]) < tol, (l, "attention", n)
        for n in host[l][1]:
            assert rel_l2(gm_t[l][n].cpu().numpy(), grads[l][1][n]) < tol, (l, "moe", n)
    return st, host, cfg


def test_three_fp32_blocks_against_the_oracle():
    acfg = AttnConfig("a", batch=2, seq_len=40, d_model=64, n_heads=4, n_kv_heads=2, weight_dtype="f32", rope_theta=1e4)
    mcfg = BlockConfig("m", tokens=80, d_model=64, n_experts=8, top_k=2, d_expert=32, d_shared=16, weight_dtype="f32")
    _run(acfg, mcfg, 3, 0.1, 2e-4)


def test_two_iterations_and_in_place_block_inverse():
    acfg = AttnConfig("a", batch=1, seq_len=24, d_model=64, n_heads=2, n_kv_heads=2, weight_dtype="f32", rope_theta=1e4)
    mcfg = BlockConfig("m", tokens=24, d_model=64, n_experts=4, top_k=2, d_expert=32, d_shared=0, weight_dtype="f32")
    st, host, cfg = _run(acfg, mcfg, 2, 0.1, 2e-4, iters=2)
    # one block's inverse pass, in place, with more than one iteration (goes through the spare stream)
    s = make_attn_streams(acfg, 9)
    pa, pm = host[0]
    Y1, Y2, info = blk.forward(pa, pm, s["x1"], s["x2"], cfg)
    a, b = dev(Y1.astype(np.float32)), dev(Y2.astype(np.float32))
    idx = dev(info["idx"].astype(np.int32))
    st.inverse_block(0, a, b, a, b, idx, inverse_iters=3)
    R1, R2 = blk.inverse(pa, pm, Y1.astype(np.float32), Y2.astype(np.float32), cfg, n_iter=3, route_override=info["idx"])
    assert rel_l2(Y1 - a.cpu().numpy(), Y1 - R1) < 2e-4 and rel_l2(Y2 - b.cpu().numpy(), Y2 - R2) < 2e-4
    assert rel_l2(a.cpu().numpy(), s["x1"]) < 1e-3 and rel_l2(b.cpu().numpy(), s["x2"]) < 1e-5


@pytest.mark.parametrize("simt", [False, True], ids=["tcgen05", "cuda_cores"])
def test_two_bf16_blocks_against_the_oracle(simt):
    import paper_2512_20920_b200 as rv
    acfg = AttnConfig("a", batch=2, seq_len=192, d_model=256, n_heads=2, n_kv_heads=1, weight_dtype="bf16")
    mcfg = BlockConfig("m", tokens=384, d_model=256, n_experts=8, top_k=2, d_expert=128, d_shared=128, weight_dtype="bf16")
    # bf16 intermediates through four branches in a row: the path's 2e-2 per branch compounds
    _run(acfg, mcfg, 2, 0.05, 3e-2, flags=rv.FLAG_FORCE_SIMT if simt else 0, moe_scale=3.0)


def test_mismatched_descriptors_are_rejected():
    import paper_2512_20920_b200 as rv
    d = rv.BlockDesc(rv.AttnDesc(2, 40, 64, 4, 2, rv.F32, 1e-6, 1e4, 32, 0),
                     rv.Desc(81, 64, 8, 2, 32, 0, rv.F32, rv.NORM_RMS, 1e-6, 32, 0), 1)
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_block_workspace_size(d)
    assert e.value.code == -2


def test_stage_one_trains_only_the_adapters():
    """Sec. 3.3, stage 1: every pre-trained weight is frozen; only the adapters' gradients are written, and they
    equal the ones of a backward pass that computes everything."""
    acfg = AttnConfig("a", batch=1, seq_len=24, d_model=64, n_heads=2, n_kv_heads=2, weight_dtype="f32", rope_theta=1e4)
    mcfg = BlockConfig("m", tokens=24, d_model=64, n_experts=4, top_k=2, d_expert=32, d_shared=0, weight_dtype="f32")
    st, host, cfg, dev_a, dev_m = _make(acfg, mcfg, 2, 0.1)
    s = make_attn_streams(acfg, 11)

    def run(stage):
        a, b, g1, g2 = dev(s["x1"]), dev(s["x2"]), dev(s["dy1"]), dev(s["dx2"])
        st.forward(a, b)
        ga_t = [{n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()} for w in dev_a]
        gm_t = [{n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()} for w in dev_m]
        ga, gm = st.grads_arrays(ga_t, gm_t, stage=stage)
        st.backward(a, b, g1, g2, ga, gm)
        assert st.status() == 0
        return ga_t, gm_t, g1, g2

    full_a, full_m, f1, f2 = run(None)
    s1_a, s1_m, h1, h2 = run(1)
    assert torch.equal(f1, h1) and torch.equal(f2, h2)            # the stream gradients do not depend on the mask
    for l in range(2):
        for grads, full in ((s1_a[l], full_a[l]), (s1_m[l], full_m[l])):
            for n, t in grads.items():
                if n in ("w_up", "w_down"):
                    assert torch.equal(t, full[n]), (l, n)
                else:
                    assert torch.isnan(t).all(), (l, n)           # never touched
