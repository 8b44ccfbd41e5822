"""The synthetic inputs have the shapes, value distributions and routing
structure the benchmark configurations state."""
import numpy as np

from oracle import revffn_oracle as orc
from workloads import CONFIGS, make_streams, make_weights, weight_shapes


def test_c0_shapes_and_distributions():
    cfg = CONFIGS["C0"]
    w, s = make_weights(cfg, 0), make_streams(cfg, 0)
    assert {n: v.shape for n, v in w.items()} == weight_shapes(cfg)
    assert "ws_gate" not in w and "b_router" not in w
    assert s["y1"].shape == (64, 64) and s["y1"].dtype == np.float32
    assert abs(s["y1"].std() - 1.0) < 0.05
    assert abs(w["w_gate"].std() - 0.02) < 0.002
    assert abs(w["norm_gamma"].mean() - 1.0) < 0.02
    w2 = make_weights(cfg, 0)
    assert all(np.array_equal(w[n], w2[n]) for n in w)
    assert not np.array_equal(make_weights(cfg, 1)["w_up"], w["w_up"])


def test_bf16_weights_are_bf16_representable():
    cfg = CONFIGS["C1"]
    w = make_weights(cfg, 0, only={"w_up", "w_router", "ws_sgate"})
    for v in w.values():
        bits = v.view(np.uint32)
        assert (bits & 0xFFFF == 0).all()


def test_zipf_bias_skews_load_with_slope_and_two_empty_experts():
    cfg = CONFIGS["C2"]
    w = make_weights(cfg, 0, only={"norm_gamma", "w_up", "w_router", "b_router"})
    y = make_streams(cfg, 0)["y1"][:4096]
    n, _ = orc.norm_fwd(y, w["norm_gamma"], cfg.norm_eps)
    u = n @ w["w_up"].astype(np.float64).T
    idx = orc.topk_indices(orc.router_logits(u, w), cfg.top_k)
    cnt = np.sort(np.bincount(idx.ravel(), minlength=cfg.n_experts))[::-1].astype(float)
    assert (cnt == 0).sum() == 2
    ranks = np.arange(1, cfg.n_experts + 1)
    sel = (ranks >= 2) & (ranks <= 40)
    slope = np.polyfit(np.log(ranks[sel]), np.log(cnt[sel]), 1)[0]
    assert abs(slope + cfg.zipf_s) < 0.1
    assert cnt[0] > 20 * cnt[50]


def test_attention_inputs_have_the_stated_shapes_and_distributions():
    from workloads.generate import ATTN_CONFIGS, attn_weight_shapes, make_attn_streams, make_attn_weights
    a0, a1 = ATTN_CONFIGS["A0"], ATTN_CONFIGS["A1"]
    assert (a1.batch, a1.seq_len, a1.d_model, a1.n_heads, a1.n_kv_heads, a1.head_dim) == (4, 2048, 2048, 16, 16, 128)
    assert a1.tokens == CONFIGS["C1"].tokens and a1.d_model == CONFIGS["C1"].d_model     # the same token batch as C1
    w, s = make_attn_weights(a0, 0), make_attn_streams(a0, 0)
    assert {n: v.shape for n, v in w.items()} == attn_weight_shapes(a0)
    assert w["w_k"].shape == (a0.n_kv_heads * a0.head_dim, a0.d_model) and w["b_k"].shape == (a0.n_kv_heads * a0.head_dim,)
    assert s["x1"].shape == (a0.tokens, a0.h) and s["x1"].dtype == np.float32
    assert set(s) == {"x1", "x2", "dy1", "dx2"} and not np.array_equal(s["x1"], s["x2"])
    assert abs(s["x2"].std() - 1.0) < 0.05 and abs(w["norm_gamma"].mean() - 1.0) < 0.02
    w2 = make_attn_weights(a0, 0)
    assert all(np.array_equal(w[n], w2[n]) for n in w)                 # seeded
    assert not np.array_equal(make_attn_weights(a0, 1)["w_q"], w["w_q"])
    # bf16 configurations: matrices exactly representable in bf16, biases and the norm scale stay fp32
    from dataclasses import replace
    wb = make_attn_weights(replace(a0, weight_dtype="bf16"), 0)
    assert (wb["w_q"].view(np.uint32) & 0xFFFF == 0).all() and (wb["w_up"].view(np.uint32) & 0xFFFF == 0).all()
    assert (wb["b_q"].view(np.uint32) & 0xFFFF != 0).any()
