"""The allocation-free routing entry point against the regular forward pass and the oracle.

revffn_moe_route_noalloc serves callers that cannot hand the library a
workspace (no cudaMalloc where they sit: allocation-free stream regions,
plug-ins that only see their inputs and outputs).  Its scratch is a fixed array
inside the library, shared by every call on the device, so the test makes two
calls in a row on different inputs and checks each against what
revffn_moe_forward selects and weighs for the same tokens, and against the
oracle's routing.  Further cases: the Qwen-shaped router (60 experts,
(E+1)*h just under the scratch limit) and the flag the entry point does not
support.  Collected last on purpose: a run
that stops at the first failure has by then run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, make_block

pytestmark = pytest.mark.gpu


def _case(seed, tokens):
    cfg = BlockConfig("noalloc", tokens=tokens, d_model=256, n_experts=12, top_k=3, d_expert=128, d_shared=128,
                      weight_dtype="bf16")
    w = make_weights(cfg, seed)
    for n in w:
        if n != "norm_gamma":
            w[n] = to_bf16_values(w[n] * 4.0)
    return cfg, w, make_streams(cfg, seed)


def _oracle_routing(cfg, w, y1):
    n, _ = orc.norm_fwd(y1, w["norm_gamma"], cfg.norm_eps)
    u = n @ w["w_up"].astype(np.float64).T
    L = orc.router_logits(u, w)
    idx = orc.topk_indices(L, cfg.top_k)
    sg = orc.sigmoid(u @ w["ws_sgate"].astype(np.float64)) if cfg.d_shared > 0 else np.zeros(len(y1))
    return L, idx, orc.topk_margin(L, cfg.top_k), sg


def _check_against_oracle(cfg, w, y1_host, idx, gates, sgate):
    L, idx_ref, margin, sg_ref = _oracle_routing(cfg, w, y1_host)
    idx = idx.cpu().numpy()
    same = (np.sort(idx, 1) == np.sort(idx_ref, 1)).all(1)
    assert (same | (margin < 1e-6)).all()                                 # index sets exact outside near-ties
    top = -np.sort(-L, axis=1)[:, : cfg.top_k + 1]
    clear = np.min(-np.diff(top, axis=1), axis=1) >= 1e-9
    assert (idx[clear] == idx_ref[clear]).all()                           # slot order too
    assert np.allclose(gates.cpu().numpy()[same], orc.gate_weights(L, idx)[same], atol=2e-6)
    assert np.allclose(sgate.cpu().numpy(), sg_ref, atol=2e-6)


def test_route_noalloc_matches_forward_on_two_calls_in_a_row():
    import paper_2512_20920_b200 as rv
    results = []
    for seed, tokens in ((0, 333), (1, 200)):           # second call reuses the same fixed scratch
        cfg, w, s = _case(seed, tokens)
        blk = make_block(cfg, w)
        y1, x2 = dev(s["y1"]), dev(s["x2"])
        idx = torch.full((tokens, cfg.top_k), -1, dtype=torch.int32, device="cuda")
        gates = torch.full((tokens, cfg.top_k), float("nan"), device="cuda")
        sgate = torch.full((tokens,), float("nan"), device="cuda")
        rv.revffn_moe_route_noalloc(blk.desc, blk.w, y1, idx, gates, sgate)
        torch.cuda.synchronize()
        results.append((cfg, blk, y1, x2, idx, gates, sgate))
        _check_against_oracle(cfg, w, s["y1"], idx, gates, sgate)
    # reference: the existing entry point, run afterwards so it cannot have primed anything
    for cfg, blk, y1, x2, idx, gates, sgate in results:
        idx_ref = torch.empty_like(idx)
        blk.forward(y1, x2, topk_idx_out=idx_ref)
        assert blk.status() == 0
        n = cfg.tokens * cfg.top_k
        gates_ref = blk.buffer("gates", torch.float32)[:n].view(cfg.tokens, cfg.top_k)
        sgate_ref = blk.buffer("sgate", torch.float32)[: cfg.tokens]
        assert torch.equal(idx, idx_ref)                                  # routing indices: bit-exact
        assert torch.allclose(gates, gates_ref, rtol=0, atol=1e-6)
        assert torch.allclose(sgate, sgate_ref, rtol=0, atol=1e-6)
        assert torch.allclose(gates.sum(1), torch.ones(cfg.tokens, device="cuda"), atol=1e-5)


def test_route_noalloc_at_the_benchmark_router_shape():
    """60 experts over 1024-wide streams: (E+1)*h = 62464 of the 65536 scratch elements.  Two calls in a row,
    against the oracle and forward."""
    import paper_2512_20920_b200 as rv
    base = CONFIGS["C1"]
    for seed, tokens in ((0, 1000), (1, 777)):
        cfg = BlockConfig("noalloc-c1", tokens=tokens, d_model=base.d_model, n_experts=base.n_experts, top_k=base.top_k,
                          d_expert=128, d_shared=128, weight_dtype="bf16")
        w, s = make_weights(cfg, seed), make_streams(cfg, seed)
        blk = make_block(cfg, w)
        y1, x2 = dev(s["y1"]), dev(s["x2"])
        idx = torch.full((tokens, cfg.top_k), -1, dtype=torch.int32, device="cuda")
        gates = torch.full((tokens, cfg.top_k), float("nan"), device="cuda")
        sgate = torch.full((tokens,), float("nan"), device="cuda")
        rv.revffn_moe_route_noalloc(blk.desc, blk.w, y1, idx, gates, sgate)
        torch.cuda.synchronize()
        _check_against_oracle(cfg, w, s["y1"], idx, gates, sgate)
        idx_ref = torch.empty_like(idx)
        blk.forward(y1, x2, topk_idx_out=idx_ref)
        assert blk.status() == 0
        # the two entry points sum the folded router in different orders (fp64 rounding): identical sets
        # except where two logits tie to that rounding
        differ = (idx.sort(1).values != idx_ref.sort(1).values).any(1)
        assert int(differ.sum()) == 0 or (_oracle_routing(cfg, w, s["y1"])[2][differ.cpu().numpy()] < 1e-9).all()
        gates_ref = blk.buffer("gates", torch.float32)[: tokens * cfg.top_k].view(tokens, cfg.top_k)
        assert torch.allclose(gates[~differ], gates_ref[~differ], rtol=0, atol=1e-6)


def test_route_noalloc_refuses_the_gating_it_cannot_compute():
    import paper_2512_20920_b200 as rv
    cfg, w, s = _case(2, 64)
    blk = make_block(cfg, w, flags=rv.FLAG_GATE_SOFTMAX_ALL)
    y1 = dev(s["y1"])
    idx = torch.zeros(64, cfg.top_k, dtype=torch.int32, device="cuda")
    g = torch.zeros(64, cfg.top_k, device="cuda")
    sg = torch.zeros(64, device="cuda")
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_moe_route_noalloc(blk.desc, blk.w, y1, idx, g, sg)
    assert e.value.code == rv.ERR_UNSUPPORTED
    assert float(g.abs().max()) == 0.0                                    # nothing was launched


def test_route_noalloc_rejects_problems_beyond_its_scratch():
    import paper_2512_20920_b200 as rv
    cfg = BlockConfig("big", tokens=8, d_model=4096, n_experts=60, top_k=4, d_expert=128, d_shared=0,
                      weight_dtype="bf16")                                # (E+1)*h = 124928 > 65536
    w = {n: np.zeros(s, dtype=np.float32) for n, s in
         dict(norm_gamma=(2048,), w_up=(4096, 2048), w_down=(2048, 4096), w_router=(60, 4096),
              w_gate=(60, 128, 4096), w_upx=(60, 128, 4096), w_downx=(60, 4096, 128)).items()}
    blk = make_block(cfg, w)
    y1 = torch.zeros(8, 2048, device="cuda")
    idx = torch.zeros(8, 4, dtype=torch.int32, device="cuda")
    g = torch.zeros(8, 4, device="cuda")
    sg = torch.zeros(8, device="cuda")
    with pytest.raises(rv.RevffnError) as e:
        rv.revffn_moe_route_noalloc(blk.desc, blk.w, y1, idx, g, sg)
    assert e.value.code == -9
    assert "scratch" in str(e.value)
