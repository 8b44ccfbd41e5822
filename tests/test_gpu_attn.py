"""Parity of the attention coupling branch (Eq. 1, its fixed-point inverse, its backward) between the
CUDA library, called through the C ABI, and the CPU oracle, on the same seeded inputs.

Tolerances: fp32 weights run every product in fp32, so only summation order differs (1e-4 relative
L2, set by the fp32 softmax and the length of the sums); bf16 weights take the path's stated 2e-2 for
outputs and gradients (bf16 operands, fp32 accumulation, P and dS rounded to bf16)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import revffn_attn_oracle as orc
from workloads.generate import ATTN_CONFIGS, AttnConfig, make_attn_streams, make_attn_weights

from helpers import dev, rel_l2

pytestmark = pytest.mark.gpu

F32_ALWAYS = ("norm_gamma", "b_q", "b_k", "b_v")


def _branch(cfg: AttnConfig, w: dict, flags: int = 0, ld_stream=None):
    import paper_2512_20920_b200 as rv
    wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
    dw = {n: torch.from_numpy(np.ascontiguousarray(v)).to(device="cuda", dtype=torch.float32 if n in F32_ALWAYS else wdt)
          for n, v in w.items() if v is not None}
    return rv.AttnBranch(batch=cfg.batch, seq_len=cfg.seq_len, d_model=cfg.d_model, n_heads=cfg.n_heads,
                         n_kv_heads=cfg.n_kv_heads, weight_dtype=rv.BF16 if cfg.weight_dtype == "bf16" else rv.F32,
                         weights=dw, norm_eps=cfg.norm_eps, rope_theta=cfg.rope_theta, flags=flags, ld_stream=ld_stream)


def _oracle_args(cfg):
    return dict(S=cfg.seq_len, n_heads=cfg.n_heads, n_kv_heads=cfg.n_kv_heads, eps=cfg.norm_eps, theta=cfg.rope_theta)


def _run_all(cfg: AttnConfig, tol: float, flags: int = 0, std: float = 0.02, seed: int = 0, n_iter=(1, 3)):
    w = make_attn_weights(cfg, seed, std=std, bias_std=std)
    s = make_attn_streams(cfg, seed)
    br = _branch(cfg, w, flags)
    oa = _oracle_args(cfg)
    x1, x2, dy1, dx2_0 = dev(s["x1"]), dev(s["x2"]), dev(s["dy1"]), dev(s["dx2"])

    # forward
    y1 = br.forward(x1, x2)
    assert br.status() == 0
    Y1 = orc.forward(w, s["x1"], s["x2"], **oa)
    A = Y1 - s["x1"]
    assert rel_l2(y1.cpu().numpy() - s["x1"], A) < tol, "branch output"

    # inverse from the oracle's Y1 (same input on both sides), several iteration counts
    y1_ref = dev(Y1.astype(np.float32))
    for n in n_iter:
        xh = br.inverse(y1_ref, x2, n_iter=n)
        assert br.status() == 0
        Xh = orc.inverse(w, Y1.astype(np.float32), s["x2"], n_iter=n, **oa)
        # compare the subtracted branch, not the stream it is subtracted from
        assert rel_l2(Y1 - xh.cpu().numpy(), Y1 - Xh) < tol, f"inverse, {n} iterations"
    assert torch.equal(br.inverse(y1_ref, x2, n_iter=0), y1_ref)

    # backward
    grads = {n: torch.full(v.shape, float("nan"), dtype=torch.float32, device="cuda") for n, v in w.items()}
    dx2 = dx2_0.clone()
    dx1 = br.backward(x1, x2, dy1, dx2, grads=grads)
    assert br.status() == 0
    dX1, dX2, G = orc.backward(w, s["x1"], s["x2"], s["dy1"], **oa)
    assert rel_l2(dx1.cpu().numpy() - s["dy1"], dX1 - s["dy1"]) < tol, "dX1 through the branch"
    assert rel_l2(dx2.cpu().numpy() - s["dx2"], dX2) < tol, "dX2 (added to the caller's gradient)"
    for n in w:
        assert rel_l2(grads[n].cpu().numpy(), G[n]) < tol, f"gradient of {n}"
    return br, w, s, grads


def test_tiny_fp32_branch_with_grouped_kv_heads_and_ragged_length():
    _run_all(ATTN_CONFIGS["A0"], 1e-4, std=0.2)


def test_tiny_fp32_branch_single_position_and_full_heads():
    cfg = replace(ATTN_CONFIGS["A0"], seq_len=1, batch=3, n_kv_heads=4)
    _run_all(cfg, 1e-4, std=0.2, n_iter=(1,))


@pytest.mark.parametrize("simt", [False, True], ids=["tcgen05", "cuda_cores"])
def test_bf16_branch_ragged_length_grouped_kv_heads(simt):
    import paper_2512_20920_b200 as rv
    cfg = AttnConfig("a", batch=2, seq_len=200, d_model=512, n_heads=4, n_kv_heads=2, weight_dtype="bf16")
    _run_all(cfg, 2e-2, flags=rv.FLAG_FORCE_SIMT if simt else 0, std=0.05)


def test_bf16_branch_whole_tiles_peaked_attention():
    cfg = AttnConfig("b", batch=3, seq_len=256, d_model=256, n_heads=2, n_kv_heads=2, weight_dtype="bf16")
    # with weights this large the branch is no contraction: repeated iterations amplify rounding
    # differences between the two sides, so only the paper's single iteration is compared
    _run_all(cfg, 2e-2, std=0.12, seed=3, n_iter=(1,))


def test_backward_accumulates_when_asked_and_skips_null_gradients():
    cfg = ATTN_CONFIGS["A0"]
    w = make_attn_weights(cfg, 1, std=0.2, bias_std=0.2)
    s = make_attn_streams(cfg, 1)
    br = _branch(cfg, w)
    x1, x2, dy1 = dev(s["x1"]), dev(s["x2"]), dev(s["dy1"])
    names = ("w_up", "w_q", "b_k", "norm_gamma")
    g1 = {n: torch.zeros(w[n].shape, dtype=torch.float32, device="cuda") for n in names}
    br.backward(x1, x2, dy1, torch.zeros_like(x2), grads=g1)
    g2 = {n: torch.full(w[n].shape, 2.0, dtype=torch.float32, device="cuda") for n in names}
    br.backward(x1, x2, dy1, torch.zeros_like(x2), grads=g2, accumulate=True)
    for n in names:
        assert torch.allclose(g2[n], g1[n] + 2.0, rtol=1e-5, atol=1e-6), n
    # dx1 may alias dy1
    ref = br.backward(x1, x2, dy1, torch.zeros_like(x2))
    buf = dy1.clone()
    out = br.backward(x1, x2, buf, torch.zeros_like(x2), dx1=buf)
    assert out.data_ptr() == buf.data_ptr() and torch.equal(buf, ref)


def test_strided_streams_and_bad_arguments():
    import paper_2512_20920_b200 as rv
    cfg = ATTN_CONFIGS["A0"]
    w = make_attn_weights(cfg, 2, std=0.2)
    s = make_attn_streams(cfg, 2)
    # both streams as views into one interleaved [T, d] tensor
    H = torch.from_numpy(np.concatenate([s["x1"], s["x2"]], axis=1)).cuda()
    br = _branch(cfg, w, ld_stream=cfg.d_model)
    out = torch.zeros_like(H)
    br.forward(H[:, :cfg.h], H[:, cfg.h:], out[:, :cfg.h])
    Y1 = orc.forward(w, s["x1"], s["x2"], **_oracle_args(cfg))
    assert rel_l2(out[:, :cfg.h].cpu().numpy() - s["x1"], Y1 - s["x1"]) < 1e-4
    assert not out[:, cfg.h:].any()
    with pytest.raises(rv.RevffnError):
        y = dev(s["x1"])
        _branch(cfg, w).inverse(y, dev(s["x2"]), x1=y, n_iter=2)       # in place with more than one iteration
    with pytest.raises(rv.RevffnError):
        rv.revffn_attn_workspace_size(rv.AttnDesc(2, 8, 64, 3, 1, rv.F32, 1e-6, 1e4, 32, 0))   # heads do not divide d
    empty = replace(cfg, batch=0)
    brz = _branch(empty, w)
    z = torch.empty(0, cfg.h, device="cuda")
    brz.forward(z, z, z)
    assert brz.status() == 0


def test_backward_reuses_the_key_value_side_of_the_inverse_pass():
    """Reversible back-propagation runs a block's inverse pass right before its gradient pass; with the
    reuse flag the gradient pass takes keys and values from the workspace.  Same arithmetic, same bits."""
    cfg = AttnConfig("r", batch=2, seq_len=200, d_model=256, n_heads=2, n_kv_heads=1, weight_dtype="bf16")
    w = make_attn_weights(cfg, 4, std=0.05, bias_std=0.05)
    s = make_attn_streams(cfg, 4)
    br = _branch(cfg, w)
    x1, x2, dy1 = dev(s["x1"]), dev(s["x2"]), dev(s["dy1"])
    names = ("w_k", "w_v", "b_k", "w_up", "norm_gamma", "w_q")
    mk = lambda: {n: torch.zeros(w[n].shape, dtype=torch.float32, device="cuda") for n in names}
    g_a, g_b = mk(), mk()
    dx2_a, dx2_b = torch.zeros_like(x2), torch.zeros_like(x2)
    y1 = br.forward(x1, x2)
    dx1_a = br.backward(x1, x2, dy1, dx2_a, grads=g_a)
    # inverse pass (leaves keys and values behind), then the gradient pass at the same x1 with the flag
    br.inverse(y1, x2, n_iter=1)
    dx1_b = br.backward(x1, x2, dy1, dx2_b, grads=g_b, reuse_kv=True)
    assert br.status() == 0
    assert torch.equal(dx1_a, dx1_b) and torch.equal(dx2_a, dx2_b)
    for n in names:
        assert torch.equal(g_a[n], g_b[n]), n
