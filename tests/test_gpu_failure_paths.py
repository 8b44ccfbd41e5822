"""The library's failure detection, exercised without faulting the GPU.

  * a bounded device-side wait that runs out: the load warp of one small matrix
    product is told to issue nothing, so the wait for its operands expires; the
    kernel must raise REVFFN_ERR_DEVICE_WAIT, free its tensor memory and return,
    and the same product must run correctly afterwards;
  * expert indices out of range in a caller-supplied expert set: reported in the
    status word, never used as an address;
  * the status word of a chain of calls on one workspace (the stack): the first
    error survives the calls that follow;
  * the debug checks: guard zones between the workspace's buffers, and the
    non-finite-logit check of the router.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from workloads import BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, grad_buffers, make_block, rel_l2, to_device_weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def _cfg(**kw):
    base = dict(name="F", tokens=300, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=256, weight_dtype="bf16")
    base.update(kw)
    return BlockConfig(**base)


def _weights(cfg, seed):
    w = make_weights(cfg, seed)
    for n in w:
        if n not in ("norm_gamma", "b_router"):
            w[n] = to_bf16_values(w[n] * 4.0)
    return w


def test_a_wait_that_runs_out_is_reported_and_the_context_survives(rv):
    from paper_2512_20920_b200.binding import DbgGemmArgs
    M, N, K = 256, 256, 256
    g = torch.Generator("cuda").manual_seed(5)
    A = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    B = torch.randn(N, K, device="cuda", generator=g).to(torch.bfloat16)
    out = torch.zeros(M, N, device="cuda", dtype=torch.bfloat16)
    status = torch.zeros(64, dtype=torch.int32, device="cuda")

    def run(**extra):
        a = DbgGemmArgs()
        a.resid_sign = 1.0
        a.M, a.N, a.K, a.lda, a.ldb, a.ldc = M, N, K, K, K, N
        a.A, a.B0, a.C = A.data_ptr(), B.data_ptr(), out.data_ptr()
        a.no_pair = 1
        for k, v in extra.items():
            setattr(a, k, v)
        status.zero_()
        code = rv.lib.revffn_dbg_gemm(C.byref(a), status.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()          # returns: the kernel left on its own
        return code, int(status[0])

    # nothing loads the operands, every wait is bounded to about a millisecond
    code, st = run(starve_operands=1, wait_cycles=2_000_000)
    assert code == 0 and st == rv.ERR_DEVICE_WAIT
    assert float(out.float().abs().max()) == 0.0           # nothing was stored
    # the hook needs the one-CTA-per-tile form
    code, _ = run(starve_operands=1, wait_cycles=2_000_000, no_pair=0)
    assert code == rv.ERR_UNSUPPORTED
    # the same product with the default bound: correct, status clean
    code, st = run()
    assert code == 0 and st == 0
    assert rel_l2(out.float().cpu().numpy(), (A.float() @ B.float().T).cpu().numpy()) <= 1e-2


def test_expert_indices_out_of_range_are_reported_not_used(rv):
    cfg = _cfg()
    w, s = _weights(cfg, 1), make_streams(cfg, 1)
    blk = make_block(cfg, w)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    y2 = blk.forward(y1, x2, topk_idx_out=idx)
    assert blk.status() == 0
    good = blk.inverse(y1, y2, topk_idx_in=idx)
    for bad_value in (-1, cfg.n_experts, 1 << 20):
        bad = idx.clone()
        bad[7, 1] = bad_value
        bad[200, 0] = bad_value
        x2b = blk.inverse(y1, y2, topk_idx_in=bad)
        assert blk.status() == rv.ERR_INDEX
        # tokens whose sets are intact are unaffected; the others lose only the bad slot
        keep = torch.ones(cfg.tokens, dtype=torch.bool, device="cuda")
        keep[7] = keep[200] = False
        assert torch.equal(x2b[keep], good[keep])
        assert torch.isfinite(x2b).all()
        dy1 = torch.zeros_like(y1)
        blk.backward(y1, dy2, dy1, grad_buffers(cfg, w), topk_idx_in=bad)
        assert blk.status() == rv.ERR_INDEX
        assert torch.isfinite(dy1).all()
    # a routing record with a bad index takes the same path (no router kernel runs there)
    rec_blk = make_block(cfg, w, flags=rv.FLAG_ROUTING_RECORD)
    rec = torch.zeros(rv.revffn_moe_routing_record_bytes(rec_blk.desc), dtype=torch.uint8, device="cuda")
    rec_blk.forward(y1, x2, topk_idx_out=rec)
    rec[: 4].view(torch.int32)[0] = cfg.n_experts + 3
    rec_blk.inverse(y1, y2, topk_idx_in=rec)
    assert rec_blk.status() == rv.ERR_INDEX
    # and a clean call afterwards clears the word
    blk.inverse(y1, y2, topk_idx_in=idx)
    assert blk.status() == 0


def test_the_first_error_of_a_chain_of_calls_survives(rv):
    """Three layers on one workspace; only the MIDDLE layer's expert sets are bad.  The layers that run after
    it are clean, and the status word must still name the error when the sweep is over."""
    cfg = _cfg(tokens=150)
    L = 3
    ws_host = [_weights(cfg, 10 + l) for l in range(L)]
    weights = [to_device_weights(cfg, w) for w in ws_host]
    stk = rv.Stack(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k,
                   d_expert=cfg.d_expert, d_shared=cfg.d_shared, weight_dtype=rv.BF16, weights=weights)
    s = make_streams(cfg, 3)
    a, b = dev(s["y1"]), dev(s["x2"])
    idx = torch.empty(L, cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    stk.forward(a, b, idx)
    assert stk.status() == 0
    ga, gb = dev(s["dy2"]), dev(s["dy2"])
    gbuf = {"w_up": torch.empty(cfg.d_model, cfg.h, device="cuda")}
    bad = idx.clone()
    bad[1, 5, 0] = cfg.n_experts
    a2, b2 = a.clone(), b.clone()
    stk.backward(a2, b2, ga.clone(), gb.clone(), stk.grads_array([gbuf] * L), topk_idx=bad)
    assert stk.status() == rv.ERR_INDEX            # layer 0 ran after layer 1 and did not erase it
    stk.backward(a, b, ga, gb, stk.grads_array([gbuf] * L), topk_idx=idx)
    assert stk.status() == 0
    # single calls: the flag keeps a word that is already set, a call without it clears the word
    blk = make_block(cfg, ws_host[0])
    y1, x2 = dev(s["y1"]), dev(s["x2"])
    blk.ws[:4].view(torch.int32)[0] = rv.ERR_DEVICE_WAIT
    blk.forward(y1, x2, flags=rv.FLAG_KEEP_STATUS)
    assert blk.status() == rv.ERR_DEVICE_WAIT
    blk.forward(y1, x2)
    assert blk.status() == 0


def test_debug_checks_guard_zones_and_non_finite_logits(rv):
    cfg = _cfg(tokens=260)
    w, s = _weights(cfg, 2), make_streams(cfg, 2)
    plain = make_block(cfg, w)
    blk = make_block(cfg, w, flags=rv.FLAG_DEBUG_CHECKS)
    assert blk.bwd_bytes > plain.bwd_bytes and blk.fwd_bytes > plain.fwd_bytes      # room for the guard zones
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    y2 = blk.forward(y1, x2)
    assert blk.status() == 0
    assert torch.equal(y2, plain.forward(y1, x2))                                    # same results with the checks on
    x2r = blk.inverse(y1, y2, save=True)
    dy1, g = torch.zeros_like(y1), grad_buffers(cfg, w)
    blk.backward(y1, dy2, dy1, g, reuse=True)
    assert blk.status() == 0                                                         # no kernel wrote past its buffer
    dy1_p, g_p = torch.zeros_like(y1), grad_buffers(cfg, w)
    plain.backward(y1, dy2, dy1_p, g_p)
    assert torch.equal(dy1, dy1_p) and all(torch.equal(g[n], g_p[n]) for n in g)
    # overwrite one byte of a guard zone by hand: the check names it
    n_zones = 0
    while True:
        try:
            off, nbytes = rv.ws_lookup(blk.desc, f"guard{n_zones}")
        except rv.RevffnError:
            break
        assert nbytes == 256 and off % 256 == 0
        n_zones += 1
    assert n_zones >= 40
    rv.revffn_dbg_check_guards(blk.desc, blk.ws)
    assert blk.status() == 0
    off, _ = rv.ws_lookup(blk.desc, "guard9")
    blk.ws[off + 17] ^= 0xFF
    rv.revffn_dbg_check_guards(blk.desc, blk.ws)
    assert blk.status() == rv.ERR_CANARY
    with pytest.raises(rv.RevffnError):
        rv.revffn_dbg_check_guards(plain.desc, plain.ws)                             # no guard zones without the flag
    # a NaN in one token's stream reaches the router's logits: reported, and the call still completes
    y1n = y1.clone()
    y1n[11, 3] = float("nan")
    out = blk.forward(y1n, x2)
    assert blk.status() == rv.ERR_NONFINITE
    ok = torch.ones(cfg.tokens, dtype=torch.bool, device="cuda")
    ok[11] = False
    assert torch.equal(out[ok], y2[ok])                                              # the other tokens are untouched
    plain.forward(y1n, x2)
    assert plain.status() == 0                                                       # without the flag nobody looks
