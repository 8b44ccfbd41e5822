"""FP8 (e4m3) routed experts, forward and inverse, against the oracle evaluated with the same quantisation.

Both sides round the same fp32 value x * (1 / scale) to e4m3 (the decision is taken in the kernels' precision), and for the
weights, whose bytes are identical on both sides, codes and scales must equal the oracle's quantiser bit for bit.
The activations are not identical on both sides: the kernels' u comes from a bf16-rounded n and an fp32
accumulation, the oracle's from fp64, so about 2^-9 of relative difference reaches the quantiser, and a value
that sits within that distance of a rounding boundary takes the neighbouring code.  With e4m3's relative spacing
of 2^-3..2^-4 a fraction delta/step of the elements flip by one step, an rms error of sqrt(delta * step), about
1.6 % per quantised operand and 2.3 % over the two in sequence (u, then g*H), on top of the bf16 path's own
0.5 %.  Tolerance of this variant, derived from that: 4e-2 relative L2 per tensor (twice the bf16 tolerance).
The distance to the unquantised evaluation (three bits of mantissa, about 4-5 %) is asserted to be what the
format gives, not more.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, make_block, max_block_rel_l2, rel_l2

pytestmark = pytest.mark.gpu

TOL = 2e-2          # bf16 path
TOL_FP8 = 4e-2      # this variant, see above


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def _weights(cfg, seed, scale=4.0):
    w = make_weights(cfg, seed)
    for n in w:
        if n not in ("norm_gamma", "b_router"):
            w[n] = to_bf16_values(w[n] * scale)
    return w


def test_expert_weight_codes_and_scales_equal_the_oracle_quantiser(rv):
    cfg = BlockConfig("q", tokens=16, d_model=256, n_experts=5, top_k=2, d_expert=128, d_shared=0, weight_dtype="bf16")
    w = _weights(cfg, 40)
    w["w_gate"][2, 7] = 0.0                                     # an all-zero row: scale 1, codes 0
    blk = make_block(cfg, w, flags=rv.FLAG_FP8_EXPERTS)
    q = blk.quantize_experts()
    torch.cuda.synchronize()
    for name, qn, sn in (("w_gate", "q_gate", "s_gate"), ("w_upx", "q_upx", "s_upx"), ("w_downx", "q_downx", "s_downx")):
        rows = w[name].reshape(-1, w[name].shape[-1])
        vals, scale = orc.quantize_rows_e4m3(rows)
        got = q[qn].view(torch.float8_e4m3fn).float().cpu().numpy().reshape(rows.shape)
        assert np.array_equal(q[sn].cpu().numpy().ravel(), scale), name
        assert np.array_equal(got, vals), name


@pytest.mark.parametrize("kw", [dict(), dict(tokens=517, d_shared=0, n_experts=9, top_k=3), dict(tokens=70, d_expert=384)])
def test_fp8_experts_forward_and_inverse(rv, kw):
    base = dict(name="F8", tokens=300, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=256, weight_dtype="bf16")
    base.update(kw)
    cfg = BlockConfig(**base)
    w, s = _weights(cfg, 41), make_streams(cfg, 41)
    blk = make_block(cfg, w, flags=rv.FLAG_FP8_EXPERTS)
    blk.quantize_experts()
    y1, x2 = dev(s["y1"]), dev(s["x2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    zero = torch.zeros_like(x2)
    F_gpu = blk.forward(y1, zero, topk_idx_out=idx).cpu().numpy()
    assert blk.status() == 0
    override = idx.cpu().numpy()
    F_q, info = orc.branch(w, s["y1"], cfg.top_k, cfg.norm_eps, route_override=override, fp8_experts=True)
    F_x, info_x = orc.branch(w, s["y1"], cfg.top_k, cfg.norm_eps)
    same = (np.sort(override, 1) == np.sort(info_x["idx"], 1)).all(1)
    assert (same | (info_x["margin"] < 1e-6)).all()                              # routing is not touched by the flag
    err_q, err_x = rel_l2(F_gpu, F_q), rel_l2(F_gpu, F_x)
    assert err_q <= TOL_FP8, f"against the oracle with the same quantisation: {err_q}"
    assert max_block_rel_l2(F_gpu, F_q) <= 2 * TOL_FP8                           # every token on its own (few values per row)
    assert 5e-3 < err_x < 1e-1, f"distance to the unquantised branch: {err_x}"
    # inverse: the subtracted branch is the added one, bit for bit; reconstruction to fp32 rounding
    y2 = blk.forward(y1, x2)
    assert torch.equal(blk.forward(y1, zero), -blk.inverse(y1, zero))
    assert rel_l2(blk.inverse(y1, y2).cpu().numpy(), s["x2"]) <= 1e-3
    # the bf16 evaluation of the same block is untouched by the extra weight members
    plain = make_block(cfg, w)
    assert rel_l2(plain.forward(y1, zero).cpu().numpy(), F_x) <= TOL


def test_fp8_experts_is_refused_where_it_does_not_apply(rv):
    cfg = BlockConfig("F8", tokens=64, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=0, weight_dtype="bf16")
    w, s = _weights(cfg, 42), make_streams(cfg, 42)
    blk = make_block(cfg, w, flags=rv.FLAG_FP8_EXPERTS)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    with pytest.raises(rv.RevffnError) as e:                                     # quantised weights not supplied yet
        blk.forward(y1, x2)
    assert e.value.code == -1
    blk.quantize_experts()
    blk.forward(y1, x2)
    with pytest.raises(rv.RevffnError) as e:                                     # gradients are taken on the bf16 path
        blk.backward(y1, dy2, torch.zeros_like(y1), {})
    assert e.value.code == rv.ERR_UNSUPPORTED
    for extra in (rv.FLAG_FORCE_SIMT, rv.FLAG_SAVE_ACTIVATIONS):
        with pytest.raises(rv.RevffnError) as e:
            blk.forward(y1, x2, flags=extra)
        assert e.value.code == rv.ERR_UNSUPPORTED


def test_fp8_experts_at_the_benchmark_shape(rv):
    """C1 (8192 tokens): the branch output on a token sample against the oracle with the same quantisation."""
    cfg = CONFIGS["C1"]
    w, s = make_weights(cfg, 0), make_streams(cfg, 0)
    blk = make_block(cfg, w, flags=rv.FLAG_FP8_EXPERTS)
    blk.quantize_experts()
    y1 = dev(s["y1"])
    zero = torch.zeros(cfg.tokens, cfg.h, device="cuda")
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    F_gpu = blk.forward(y1, zero, topk_idx_out=idx).cpu().numpy()
    assert blk.status() == 0 and np.isfinite(F_gpu).all()
    sample = np.sort(np.random.default_rng(3).choice(cfg.tokens, 192, replace=False))
    ov = idx.cpu().numpy()[sample]
    F_q, _ = orc.branch(w, s["y1"][sample], cfg.top_k, cfg.norm_eps, route_override=ov, fp8_experts=True)
    F_x, _ = orc.branch(w, s["y1"][sample], cfg.top_k, cfg.norm_eps, route_override=ov)
    assert rel_l2(F_gpu[sample], F_q) <= TOL_FP8
    assert 5e-3 < rel_l2(F_gpu[sample], F_x) < 1e-1
    assert torch.equal(blk.forward(y1, zero), -blk.inverse(y1, zero))
