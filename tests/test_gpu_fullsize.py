"""Full-size parity in the launch configuration the benchmark times: the
Qwen1.5-MoE-A2.7B-shaped block at 8192 tokens (near-uniform routing) and at
16384 tokens under Zipf(1.2) routing with two empty experts.

The oracle cannot afford the whole batch, so:
  * routing is checked for EVERY token (logits are cheap);
  * the branch output, the reconstruction and dY1 are checked on a seeded token
    sample (tokens are independent through this branch);
  * weight gradients use a property that holds at any size: tokens whose
    upstream gradient is zero contribute nothing, so the full-size GPU backward
    with dY2 zeroed outside a sample must equal the oracle's backward over that
    sample alone;
  * one mid-sized expert's gradients are checked with the complete dY2 (all of
    its tokens), and an empty expert's gradients must be exactly zero.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, make_streams, make_weights

from helpers import dev, make_block, rel_l2

pytestmark = pytest.mark.gpu

TOL = 2e-2
TOL_RECON = 1e-3
MARGIN = 1e-6
N_SAMPLE = 384


@pytest.mark.parametrize("name", ["C1", "C2"])
def test_full_size_block(name):
    cfg = CONFIGS[name]
    T, k, E = cfg.tokens, cfg.top_k, cfg.n_experts
    w, s = make_weights(cfg, 0), make_streams(cfg, 0)
    blk = make_block(cfg, w)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx_d = torch.empty(T, k, dtype=torch.int32, device="cuda")
    y2 = blk.forward(y1, x2, topk_idx_out=idx_d)
    assert blk.status() == 0
    idx = idx_d.cpu().numpy()

    # ---- routing, every token
    n, _ = orc.norm_fwd(s["y1"], w["norm_gamma"], cfg.norm_eps)
    u = n @ w["w_up"].astype(np.float64).T
    L = orc.router_logits(u, w)
    idx_ref, margin = orc.topk_indices(L, k), orc.topk_margin(L, k)
    same = (np.sort(idx, 1) == np.sort(idx_ref, 1)).all(1)
    bad = ~same & (margin >= MARGIN)
    assert not bad.any(), f"{bad.sum()} tokens routed differently outside the margin"
    top = -np.sort(-L, axis=1)[:, : k + 1] if k < E else -np.sort(-L, axis=1)
    clear = np.min(-np.diff(top, axis=1), axis=1) >= 1e-9
    assert (idx[clear] == idx_ref[clear]).all()           # slot order too where no two logits nearly tie
    gates = blk.buffer("gates", torch.float32)[: T * k].view(T, k).cpu().numpy()
    assert np.allclose(gates[same], orc.gate_weights(L, idx)[same], atol=2e-6)
    cnt = np.bincount(idx.ravel(), minlength=E)
    cnt_gpu = blk.buffer("expert_cnt", torch.int32)[:E].cpu().numpy()
    assert (cnt == cnt_gpu).all()
    off = blk.buffer("expert_off", torch.int32)[: E + 1].cpu().numpy()
    assert (np.diff(off) == ((cnt + 127) // 128) * 128).all()
    if cfg.zipf_s is not None:
        assert (cnt == 0).sum() >= 2 and cnt.max() > 20 * np.median(cnt[cnt > 0])

    # ---- branch output and reconstruction on a token sample
    rng = np.random.default_rng(0)
    sample = np.sort(rng.choice(T, N_SAMPLE, replace=False))
    zero = torch.zeros_like(x2)
    F_gpu = blk.forward(y1, zero).cpu().numpy()
    F_ref, _ = orc.branch(w, s["y1"][sample], k, cfg.norm_eps, route_override=idx[sample])
    assert rel_l2(F_gpu[sample], F_ref) <= TOL
    assert np.isfinite(F_gpu).all()
    x2_rec = blk.inverse(y1, y2)
    assert rel_l2(x2_rec.cpu().numpy(), s["x2"]) <= TOL_RECON
    assert torch.equal(blk.forward(y1, zero), -blk.inverse(y1, zero))

    # ---- backward, complete dY2: dY1 on the sample; one mid-sized expert; empty experts
    grads = {n_: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n_, v in w.items()}
    dy1 = torch.zeros_like(y1)
    blk.backward(y1, dy2, dy1, grads)
    assert blk.status() == 0
    ref_s = orc.backward(w, s["y1"][sample], s["dy2"][sample], k, cfg.norm_eps, route_override=idx[sample])
    assert rel_l2(dy1.cpu().numpy()[sample], ref_s["dy1"]) <= TOL
    for g in grads.values():
        assert torch.isfinite(g).all()
    mid = int(np.argmin(np.abs(cnt - 400)))
    toks = np.nonzero((idx == mid).any(1))[0]
    ref_e = orc.backward(w, s["y1"][toks], s["dy2"][toks], k, cfg.norm_eps, route_override=idx[toks])
    for name_ in ("w_gate", "w_upx", "w_downx"):
        assert rel_l2(grads[name_][mid].cpu().numpy(), ref_e[name_][mid]) <= TOL, (name_, mid, len(toks))
    assert rel_l2(grads["w_router"][mid].cpu().numpy(), ref_e["w_router"][mid]) <= TOL
    for e in np.nonzero(cnt == 0)[0]:
        for name_ in ("w_gate", "w_upx", "w_downx", "w_router"):
            assert float(grads[name_][e].abs().max()) == 0.0

    # ---- backward with dY2 zeroed outside the sample == oracle over the sample alone (all weights)
    mask = torch.zeros(T, 1, device="cuda")
    mask[torch.from_numpy(sample).cuda()] = 1.0
    dy1m = torch.zeros_like(y1)
    blk.backward(y1, dy2 * mask, dy1m, grads)
    assert blk.status() == 0
    assert float(dy1m[mask[:, 0] == 0].abs().max()) == 0.0
    for name_, g in grads.items():
        gn = g.cpu().numpy()
        if np.linalg.norm(ref_s[name_]) == 0:
            assert np.abs(gn).max() == 0, name_
        else:
            err = rel_l2(gn, ref_s[name_])
            assert err <= TOL, f"{name_} rel-L2 {err}"
