"""The allocation-free routing entry point against the regular forward pass.

revffn_moe_route_noalloc serves callers that cannot hand the library a
workspace (no cudaMalloc where they sit: allocation-free stream regions,
plug-ins that only see their inputs and outputs).  Its scratch is a fixed array
inside the library, shared by every call on the device, so the test makes two
calls in a row on different inputs and checks each against what
revffn_moe_forward selects and weighs for the same tokens.  Collected last on
purpose: a run that stops at the first failure has by then run everything else.
"""
import numpy as np
import pytest
import torch

from workloads import BlockConfig, make_streams, make_weights, to_bf16_values

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
