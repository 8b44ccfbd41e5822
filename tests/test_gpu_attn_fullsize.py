"""Full-size parity of the attention coupling branch in the launch configuration the benchmark times:
the Qwen1.5-MoE-A2.7B-shaped attention layer at 4 sequences x 2048 positions.

Sequences do not attend to each other, so the oracle evaluates ONE whole sequence (all 2048 positions,
every head) and the GPU's rows of that sequence must match it: branch output, one-iteration inverse and
dX1, dX2.  Weight gradients use a property that holds at any size: tokens whose upstream gradient is zero
contribute nothing, so the full-size GPU backward with dY1 zeroed outside that sequence must equal the
oracle's backward over that sequence alone."""
import numpy as np
import pytest
import torch

from oracle import revffn_attn_oracle as orc
from workloads.generate import ATTN_CONFIGS, make_attn_streams, make_attn_weights

from helpers import dev, rel_l2
from test_gpu_attn import _branch

pytestmark = pytest.mark.gpu

TOL = 2e-2


def test_full_size_attention_branch():
    cfg = ATTN_CONFIGS["A1"]
    S, h, b = cfg.seq_len, cfg.h, 2                      # the sequence the oracle evaluates
    w, s = make_attn_weights(cfg, 0), make_attn_streams(cfg, 0)
    br = _branch(cfg, w)
    x1, x2, dy1 = dev(s["x1"]), dev(s["x2"]), dev(s["dy1"])
    rows = slice(b * S, (b + 1) * S)
    kw = dict(S=S, n_heads=cfg.n_heads, n_kv_heads=cfg.n_kv_heads, eps=cfg.norm_eps, theta=cfg.rope_theta)

    y1 = br.forward(x1, x2)
    assert br.status() == 0
    y1_h = y1.cpu().numpy()
    assert np.isfinite(y1_h).all()
    Y1 = orc.forward(w, s["x1"][rows], s["x2"][rows], **kw)
    assert rel_l2(y1_h[rows] - s["x1"][rows], Y1 - s["x1"][rows]) <= TOL

    # inverse pass, the paper's single iteration, from the GPU's own output
    x1_rec = br.inverse(y1, x2, n_iter=1).cpu().numpy()
    X1_rec = orc.inverse(w, y1_h[rows], s["x2"][rows], n_iter=1, **kw)
    assert rel_l2(y1_h[rows] - x1_rec[rows], y1_h[rows] - X1_rec) <= TOL
    err1 = rel_l2(x1_rec, s["x1"])
    err3 = rel_l2(br.inverse(y1, x2, n_iter=3).cpu().numpy(), s["x1"])
    assert err3 < err1 < rel_l2(y1_h, s["x1"])           # every iteration brings the stream closer to the input
    assert err1 < 5e-3 and err3 < 5e-4

    # backward with the complete upstream gradient: the stream gradients of sequence b
    dX1, dX2, G = orc.backward(w, s["x1"][rows], s["x2"][rows], s["dy1"][rows], **kw)
    dx2 = torch.zeros_like(x2)
    dx1 = br.backward(x1, x2, dy1, dx2).cpu().numpy()
    assert br.status() == 0
    assert rel_l2(dx1[rows] - s["dy1"][rows], dX1 - s["dy1"][rows]) <= TOL
    assert rel_l2(dx2.cpu().numpy()[rows], dX2) <= TOL

    # backward with dY1 zero outside sequence b: every weight gradient against the oracle on that sequence
    dy1_b = torch.zeros_like(dy1)
    dy1_b[rows] = dy1[rows]
    grads = {n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()}
    dx2 = torch.zeros_like(x2)
    dx1 = br.backward(x1, x2, dy1_b, dx2, grads=grads)
    assert br.status() == 0
    for n in w:
        assert rel_l2(grads[n].cpu().numpy(), G[n]) <= TOL, n
    outside = torch.ones(cfg.tokens, dtype=torch.bool, device="cuda")
    outside[rows] = False
    assert not dx1[outside].any() and not dx2[outside].any()     # other sequences receive no gradient
