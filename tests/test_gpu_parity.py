"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the
same seeded inputs.

Tolerances (stated by the benchmark definition):
  * routing index sets: bit-exact; tokens whose oracle top-k margin is below
    1e-6 are exempt (for them the oracle is re-run with the GPU's expert set);
  * bf16 GEMM outputs (branch output F, dY1, every weight gradient): relative
    L2 <= 2e-2 per tensor; the fp32 configuration C0 is held to 1e-4;
  * reconstructed X2 against the original: relative L2 <= 1e-3.
"""
import numpy as np
import pytest
import torch

from oracle import revffn_oracle as orc
from workloads import CONFIGS, BlockConfig, make_streams, make_weights, to_bf16_values

from helpers import dev, grad_buffers, make_block, max_block_rel_l2, rel_l2

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-4
TOL_RECON = 1e-3
MARGIN = 1e-6


@pytest.fixture(scope="module")
def rv():
    import paper_2512_20920_b200 as rv
    return rv


def small_cfg(**kw):
    base = dict(name="S", tokens=300, d_model=256, n_experts=6, top_k=2, d_expert=128, d_shared=256,
                weight_dtype="bf16")
    base.update(kw)
    return BlockConfig(**base)


def scaled_weights(cfg, seed, scale):
    """Weights scaled up (and re-rounded to bf16) so that the branch output is
    O(1) even at the small test widths."""
    w = make_weights(cfg, seed)
    for n in w:
        if n not in ("norm_gamma", "b_router"):
            w[n] = w[n] * scale
            if cfg.weight_dtype == "bf16":
                w[n] = to_bf16_values(w[n])
    return w


def check_routing(idx_gpu, info, k):
    """Index sets bit-exact outside the exempt margin; returns the override to use."""
    idx_gpu = np.asarray(idx_gpu)
    same = (np.sort(idx_gpu, axis=1) == np.sort(info["idx"], axis=1)).all(axis=1)
    bad = ~same & (info["margin"] >= MARGIN)
    assert not bad.any(), f"{bad.sum()} tokens routed differently outside the {MARGIN} margin"
    return idx_gpu if (~same).any() else None


def run_all_passes(rv, cfg, w, s, tol, flags=0, norm_none=False, check_grads=True, gating="renorm"):
    if gating == "softmax_all":
        flags |= rv.FLAG_GATE_SOFTMAX_ALL
    blk = make_block(cfg, w, flags=flags, norm_none=norm_none)
    norm = "none" if norm_none else "rms"
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    y2 = blk.forward(y1, x2, topk_idx_out=idx)
    assert blk.status() == 0
    y2_ref, info = orc.forward(w, s["y1"], s["x2"], cfg.top_k, cfg.norm_eps, norm, gating=gating)
    override = check_routing(idx.cpu().numpy(), info, cfg.top_k)
    if override is not None:
        y2_ref, info = orc.forward(w, s["y1"], s["x2"], cfg.top_k, cfg.norm_eps, norm, route_override=override, gating=gating)
    # slot order too, where margins are clear
    clear = info["margin"] >= MARGIN
    gates = blk.buffer("gates", torch.float32)[: cfg.tokens * cfg.top_k].view(cfg.tokens, cfg.top_k).cpu().numpy()
    if gating == "renorm":
        assert np.allclose(gates.sum(axis=1), 1.0, atol=1e-6)
    else:
        assert (gates.sum(axis=1) < 1.0).all() or cfg.top_k == cfg.n_experts
    assert np.allclose(gates[clear], info["gates"][clear], atol=1e-5)
    # the branch output itself (X2 = 0), so that the pass-through term does not mask its error
    zero = torch.zeros_like(x2)
    f_fwd = blk.forward(y1, zero)
    err_F = rel_l2(f_fwd.cpu().numpy(), info["F"])
    assert err_F <= tol, f"F rel-L2 {err_F}"
    assert rel_l2(y2.cpu().numpy(), y2_ref) <= tol

    # inverse: reconstruct X2 from (Y1, Y2)
    x2_rec = blk.inverse(y1, y2)
    assert blk.status() == 0
    assert rel_l2(x2_rec.cpu().numpy(), s["x2"]) <= TOL_RECON
    x2_ref, _ = orc.inverse(w, s["y1"], y2.cpu().numpy(), cfg.top_k, cfg.norm_eps, norm, route_override=override, gating=gating)
    assert rel_l2(x2_rec.cpu().numpy(), x2_ref) <= tol

    # the subtracted branch is bit-identical to the added one
    f_inv = blk.inverse(y1, zero)
    assert torch.equal(f_fwd, -f_inv)

    # backward
    dy1 = torch.zeros(cfg.tokens, cfg.h, device="cuda")      # zero start: no cancellation in the comparison
    grads = grad_buffers(cfg, w) if check_grads else {}
    blk.backward(y1, dy2, dy1, grads)
    assert blk.status() == 0
    ref = orc.backward(w, s["y1"], s["dy2"], cfg.top_k, cfg.norm_eps, norm, route_override=override, gating=gating)
    err = rel_l2(dy1.cpu().numpy(), ref["dy1"])
    assert err <= tol, f"dY1 rel-L2 {err}"
    errs = {}
    for name, g in grads.items():
        gn = g.cpu().numpy()
        assert np.isfinite(gn).all(), name
        if np.linalg.norm(ref[name]) == 0:
            assert np.abs(gn).max() == 0, name
            continue
        errs[name] = rel_l2(gn, ref[name])
        assert errs[name] <= tol, f"{name} rel-L2 {errs[name]}"
        if name in ("w_gate", "w_upx", "w_downx"):      # expert by expert as well
            err_e = max_block_rel_l2(gn, ref[name])
            assert err_e <= tol, f"{name} largest per-expert rel-L2 {err_e}"
    # dY1 is accumulated into; with the accumulate flag a second call adds the same weight gradients
    if check_grads:
        before = {n: g.clone() for n, g in grads.items()}
        dy1_init = torch.randn(cfg.tokens, cfg.h, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
        dy1b = dy1_init.clone()
        blk.backward(y1, dy2, dy1b, grads, accumulate=True)
        for n, g in grads.items():
            assert torch.allclose(g, 2 * before[n], rtol=1e-5, atol=1e-7), n
        assert torch.equal(dy1b, dy1_init + dy1)
    return blk, info, errs


# ------------------------------------------------------------------ C0: tiny fp32 block
def test_c0_all_passes_fp32(rv):
    cfg = CONFIGS["C0"]
    w, s = make_weights(cfg, 0), make_streams(cfg, 0)
    run_all_passes(rv, cfg, w, s, TOL_F32)


def test_c0_scaled_weights_fp32(rv):
    cfg = CONFIGS["C0"]
    w, s = scaled_weights(cfg, 3, 5.0), make_streams(cfg, 3)
    run_all_passes(rv, cfg, w, s, TOL_F32)


# ------------------------------------------------------------------ small bf16 blocks, both GEMM back ends
@pytest.mark.parametrize("simt", [True, False])
@pytest.mark.parametrize("kw", [dict(), dict(d_shared=0, tokens=517), dict(tokens=1), dict(tokens=7, top_k=6),
                                dict(n_experts=40, top_k=4, tokens=130)])
def test_small_bf16_all_passes(rv, simt, kw):
    cfg = small_cfg(**kw)
    w, s = scaled_weights(cfg, 1, 4.0), make_streams(cfg, 1)
    run_all_passes(rv, cfg, w, s, TOL_BF16, flags=rv.FLAG_FORCE_SIMT if simt else 0)


def test_norm_none_and_router_bias(rv):
    cfg = small_cfg(tokens=200)
    w, s = scaled_weights(cfg, 2, 4.0), make_streams(cfg, 2)
    w["b_router"] = np.array([0.5, -0.5, 0.0, -40.0, 0.25, -40.0], dtype=np.float32)   # two experts never chosen
    blk, info, _ = run_all_passes(rv, cfg, w, s, TOL_BF16)
    cnt = blk.buffer("expert_cnt", torch.int32)[: cfg.n_experts].cpu().numpy()
    assert cnt[3] == 0 and cnt[5] == 0 and cnt.sum() == cfg.tokens * cfg.top_k
    run_all_passes(rv, cfg, w, s, TOL_BF16, norm_none=True)


def test_empty_batch_is_a_no_op(rv):
    cfg = small_cfg(tokens=0)
    w = scaled_weights(cfg, 1, 4.0)
    blk = make_block(cfg, w)
    e = torch.empty(0, cfg.h, device="cuda")
    blk.forward(e, e, e)
    blk.inverse(e, e, e)
    blk.backward(e, e, e, {})
    assert blk.status() == 0


def test_strided_streams_and_in_place_coupling(rv):
    """Streams as the two halves of one [T, d] tensor (row stride d); Y2 written over X2."""
    cfg = small_cfg(tokens=260)
    w, s = scaled_weights(cfg, 4, 4.0), make_streams(cfg, 4)
    blk = make_block(cfg, w, ld_stream=cfg.d_model)
    H = torch.empty(cfg.tokens, cfg.d_model, device="cuda")
    H[:, : cfg.h] = dev(s["y1"]); H[:, cfg.h:] = dev(s["x2"])
    y1v, x2v = H[:, : cfg.h], H[:, cfg.h:]
    blk.forward(y1v, x2v, x2v)
    ref, info = orc.forward(w, s["y1"], s["x2"], cfg.top_k)
    assert rel_l2(H[:, cfg.h:].cpu().numpy() - s["x2"], info["F"]) <= TOL_BF16
    assert torch.equal(H[:, : cfg.h].cpu(), torch.from_numpy(s["y1"]))
    blk.inverse(y1v, x2v, x2v)
    assert rel_l2(H[:, cfg.h:].cpu().numpy(), s["x2"]) <= TOL_RECON


def test_reuse_routing_indices(rv):
    cfg = small_cfg()
    w, s = scaled_weights(cfg, 5, 4.0), make_streams(cfg, 5)
    blk = make_block(cfg, w)
    y1, x2 = dev(s["y1"]), dev(s["x2"])
    idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
    y2 = blk.forward(y1, x2, topk_idx_out=idx)
    x2a = blk.inverse(y1, y2)
    x2b = blk.inverse(y1, y2, topk_idx_in=idx)
    assert torch.equal(x2a, x2b)
    # a forced (different) expert set is honoured
    forced = torch.tensor([[0, 1]], dtype=torch.int32, device="cuda").repeat(cfg.tokens, 1)
    x2c = blk.inverse(y1, y2, topk_idx_in=forced)
    ref, _ = orc.inverse(w, s["y1"], y2.cpu().numpy(), cfg.top_k, route_override=forced.cpu().numpy())
    assert rel_l2(x2c.cpu().numpy(), ref) <= TOL_BF16


def test_tensor_core_and_cuda_core_backends_agree(rv):
    cfg = small_cfg(tokens=400, n_experts=8, top_k=3, d_expert=256, d_shared=384, d_model=512)
    w, s = scaled_weights(cfg, 6, 3.0), make_streams(cfg, 6)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    out = {}
    for name, flags in (("tc", 0), ("simt", rv.FLAG_FORCE_SIMT)):
        blk = make_block(cfg, w, flags=flags)
        y2 = blk.forward(y1, x2)
        dy1 = torch.zeros_like(y1)
        g = grad_buffers(cfg, w)
        blk.backward(y1, dy2, dy1, g)
        assert blk.status() == 0
        out[name] = dict(y2=y2, dy1=dy1, **g)
    for n in out["tc"]:
        a, b = out["tc"][n].cpu().numpy(), out["simt"][n].cpu().numpy()
        if n == "y2":
            a, b = a - s["x2"], b - s["x2"]
        assert rel_l2(a, b) <= 5e-3, n


@pytest.mark.parametrize("simt", [True, False])
def test_backward_reuses_a_saved_evaluation(rv, simt):
    """A backward pass that reads the intermediates a forward or inverse call left in the
    workspace gives bit for bit what the recomputing backward pass gives."""
    cfg = small_cfg(tokens=333, n_experts=8, top_k=3)
    w, s = scaled_weights(cfg, 7, 4.0), make_streams(cfg, 7)
    blk = make_block(cfg, w, flags=rv.FLAG_FORCE_SIMT if simt else 0)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    y2 = blk.forward(y1, x2)
    x2_plain = blk.inverse(y1, y2)
    dy1_plain, g_plain = torch.zeros_like(y1), grad_buffers(cfg, w)
    blk.backward(y1, dy2, dy1_plain, g_plain)
    for first in ("inverse", "forward"):
        if first == "inverse":
            x2_rec = blk.inverse(y1, y2, save=True)
            assert torch.equal(x2_rec, x2_plain)
        else:
            assert torch.equal(blk.forward(y1, x2, save=True), y2)
        dy1, g = torch.zeros_like(y1), grad_buffers(cfg, w)
        blk.backward(y1, dy2, dy1, g, reuse=True)
        assert blk.status() == 0
        assert torch.equal(dy1, dy1_plain), first
        for n in g:
            assert torch.equal(g[n], g_plain[n]), (first, n)
    # a workspace of forward size is refused when the intermediates are to be kept
    small = torch.empty(blk.fwd_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(rv.RevffnError):
        blk.forward(y1, x2, save=True, ws=small)


@pytest.mark.parametrize("gating", ["renorm", "softmax_all"])
def test_all_passes_with_the_second_stream(rv, gating):
    """The tensor-core back end puts the router, the shared expert and the weight gradients on a second stream of
    the library's own (every tensor-core case in this file runs that way): the same parity at the largest size the
    oracle does in full, with both gate conventions."""
    cfg = small_cfg(tokens=1300, n_experts=7, top_k=3)
    w, s = scaled_weights(cfg, 12, 4.0), make_streams(cfg, 12)
    run_all_passes(rv, cfg, w, s, TOL_BF16, gating=gating)


@pytest.mark.parametrize("sgd", [False, True])
def test_the_second_stream_changes_no_bit(rv, sgd):
    """Every output of the three passes (recomputing and shared evaluation, gradients or the fused update) with the
    second stream equals, bit for bit, the output with every launch on the caller's stream; repeated, because a
    missing ordering between the two streams would show only now and then."""
    cfg = small_cfg(tokens=2304, n_experts=8, top_k=2, d_model=512, d_expert=256, d_shared=512)
    w, s = scaled_weights(cfg, 13, 4.0), make_streams(cfg, 13)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])

    def one_round(extra):
        blk = make_block(cfg, w)              # fresh weights: the fused update changes them
        out = {}
        out["y2"] = blk.forward(y1, x2, flags=extra)
        out["x2r"] = blk.inverse(y1, out["y2"], save=True, flags=rv.FLAG_ROUTER_FOLDED | extra)
        names = [n for n in rv.UPD_NAMES if n in blk.weights] if sgd else []
        g = {n: t for n, t in grad_buffers(cfg, w).items() if n not in names}
        dy1 = torch.zeros_like(y1)
        if sgd:
            blk.backward(y1, dy2, dy1, g, reuse=True, flags=extra, sgd=rv.make_sgd(1e-3, names))
            for n in names:
                out["W_" + n] = blk.weights[n].clone()
        else:
            blk.backward(y1, dy2, dy1, g, reuse=True, flags=extra)
            dy1b, g2 = torch.zeros_like(y1), grad_buffers(cfg, w)
            blk.backward(y1, dy2, dy1b, g2, flags=extra)          # recomputing form
            out["dy1_recomputed"] = dy1b
            for n, t in g2.items():
                out["g2_" + n] = t
        out["dy1"] = dy1
        for n, t in g.items():
            out["g_" + n] = t
        torch.cuda.synchronize()
        assert blk.status() == 0
        return out

    ref = one_round(rv.FLAG_SINGLE_STREAM)
    for _ in range(4):
        got = one_round(0)
        assert got.keys() == ref.keys()
        for n in ref:
            assert torch.equal(got[n], ref[n]), n


@pytest.mark.parametrize("two_streams,tokens", [(False, 500), (True, 500), (True, 2100)])
def test_host_step_matches_the_device_entry_points(rv, two_streams, tokens):
    """The host-buffer step (copies in, three passes, copies out; optionally with a second stream for the
    transfers) returns exactly what the three device entry points return."""
    cfg = small_cfg(tokens=tokens)      # from 2048 tokens on, the two-stream form runs the forward pass in two halves
    w, s = scaled_weights(cfg, 8, 4.0), make_streams(cfg, 8)
    blk = make_block(cfg, w)
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    y2 = blk.forward(y1, x2)
    x2r = blk.inverse(y1, y2)
    dy1, g_ref = torch.zeros_like(y1), grad_buffers(cfg, w)
    blk.backward(y1, dy2, dy1, g_ref)
    pin = lambda a: torch.from_numpy(a).pin_memory()
    hy1, hx2, hdy2 = pin(s["y1"]), pin(s["x2"]), pin(s["dy2"])
    hy2, hx2r, hdy1 = (torch.empty_like(hy1).pin_memory() for _ in range(3))
    slot = ((hy1.numel() * 4 + 255) // 256) * 256
    staging = torch.empty(6 * slot, dtype=torch.uint8, device="cuda")
    g = grad_buffers(cfg, w)
    cs = torch.cuda.Stream() if two_streams else None
    for _ in range(2):      # twice: the second step starts while the first one's copies may still be in flight
        rv.revffn_moe_step_host(blk.desc, blk.w, blk.grads_struct(g), hy1, hx2, hdy2, hy2, hx2r, hdy1, staging, blk.ws,
                                copy_stream=cs.cuda_stream if cs is not None else None)
    torch.cuda.synchronize()
    assert blk.status() == 0
    assert torch.equal(hy2, y2.cpu()) and torch.equal(hx2r, x2r.cpu()) and torch.equal(hdy1, dy1.cpu())
    for n in g:
        assert torch.equal(g[n], g_ref[n]), n


def test_pipelined_host_steps_match_the_device_entry_points(rv):
    """Five pipelined host steps on alternating inputs (the uploads of a step run beside the step before it,
    its downloads beside the step after it): every step's host outputs, read once the copy stream has passed the
    event recorded after its call, equal the device entry points' results bit for bit."""
    cfg = small_cfg(tokens=700)
    w = scaled_weights(cfg, 8, 4.0)
    blk = make_block(cfg, w)
    pin = lambda a: torch.from_numpy(a).pin_memory()
    cases = []
    for seed in (21, 22):
        s = make_streams(cfg, seed)
        y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
        y2 = blk.forward(y1, x2)
        x2r = blk.inverse(y1, y2)
        dy1, g_ref = torch.zeros_like(y1), grad_buffers(cfg, w)
        blk.backward(y1, dy2, dy1, g_ref)
        host_in = [pin(s[n]) for n in ("y1", "x2", "dy2")]
        host_out = [torch.empty_like(host_in[0]).pin_memory() for _ in range(3)]
        cases.append((host_in, host_out, [y2.cpu(), x2r.cpu(), dy1.cpu()], g_ref))
    slot = ((cases[0][0][0].numel() * 4 + 255) // 256) * 256
    staging = torch.empty(12 * slot, dtype=torch.uint8, device="cuda")
    cs = torch.cuda.Stream()
    g = grad_buffers(cfg, w)
    with pytest.raises(rv.RevffnError):                                # six slots are not enough for this form
        rv.revffn_moe_step_host(blk.desc, blk.w, blk.grads_struct(g), *cases[0][0], *cases[0][1], staging[:6 * slot], blk.ws,
                                copy_stream=cs.cuda_stream, pipelined=True)
    with pytest.raises(rv.RevffnError) as e:                           # and it needs the copy stream
        rv.revffn_moe_step_host(blk.desc, blk.w, blk.grads_struct(g), *cases[0][0], *cases[0][1], staging, blk.ws, pipelined=True)
    assert e.value.code == rv.ERR_UNSUPPORTED
    events, prev = [], None
    for i in range(5):
        host_in, host_out, ref, g_ref = cases[i & 1]
        rv.revffn_moe_step_host(blk.desc, blk.w, blk.grads_struct(g), *host_in, *host_out, staging, blk.ws,
                                copy_stream=cs.cuda_stream, pipelined=True)
        ev = torch.cuda.Event()
        ev.record(cs)
        if prev is not None:            # read the previous step's results while this one runs
            prev[0].synchronize()
            for got, want in zip(prev[1], prev[2]):
                assert torch.equal(got, want)
            for t in prev[1]:
                t.fill_(float("nan"))
        prev = (ev, host_out, ref)
    prev[0].synchronize()
    for got, want in zip(prev[1], prev[2]):
        assert torch.equal(got, want)
    torch.cuda.synchronize()
    assert blk.status() == 0
    for n in g:                          # the gradients of the last step (case 0)
        assert torch.equal(g[n], cases[0][3][n]), n


@pytest.mark.parametrize("kw", [dict(n_experts=64, top_k=8, tokens=150), dict(n_experts=130, top_k=3, tokens=97),
                                dict(n_experts=256, top_k=8, tokens=70, d_shared=0)])
def test_many_experts(rv, kw):
    """More experts than one pass of the router's logit tile holds (64 incl. the shared-gate row), up to the
    largest supported count, and the largest top-k; every weight gradient (router weights included) is compared."""
    cfg = small_cfg(**kw)
    w, s = scaled_weights(cfg, 9, 4.0), make_streams(cfg, 9)
    run_all_passes(rv, cfg, w, s, TOL_BF16)


@pytest.mark.parametrize("simt", [True, False])
@pytest.mark.parametrize("kw", [dict(), dict(n_experts=40, top_k=4, tokens=130), dict(d_shared=0, tokens=257)])
def test_gating_without_renormalisation(rv, simt, kw):
    """Gates taken from the softmax over all experts: forward, inverse and backward (where every
    logit, selected or not, now carries a gradient) against the oracle in the same mode."""
    cfg = small_cfg(**kw)
    w, s = scaled_weights(cfg, 10, 4.0), make_streams(cfg, 10)
    run_all_passes(rv, cfg, w, s, TOL_BF16, flags=rv.FLAG_FORCE_SIMT if simt else 0, gating="softmax_all")


def test_gating_without_renormalisation_fp32(rv):
    cfg = CONFIGS["C0"]
    w, s = scaled_weights(cfg, 11, 5.0), make_streams(cfg, 11)
    run_all_passes(rv, cfg, w, s, TOL_F32, gating="softmax_all")


def test_routing_record_replaces_the_router(rv):
    """A routing record written by forward carries indices, gate weights and the shared gate; inverse and
    backward given the record run no router and use exactly those values, even for a perturbed y1."""
    cfg = small_cfg(tokens=321, n_experts=8, top_k=3)
    w, s = scaled_weights(cfg, 12, 4.0), make_streams(cfg, 12)
    plain = make_block(cfg, w)
    blk = make_block(cfg, w, flags=rv.FLAG_ROUTING_RECORD)
    nrec = rv.revffn_moe_routing_record_bytes(blk.desc)
    T, k = cfg.tokens, cfg.top_k
    assert nrec % 16 == 0 and nrec >= T * (2 * k + 1) * 4
    y1, x2, dy2 = dev(s["y1"]), dev(s["x2"]), dev(s["dy2"])
    rec = torch.zeros(nrec, dtype=torch.uint8, device="cuda")
    idx = torch.empty(T, k, dtype=torch.int32, device="cuda")
    y2 = blk.forward(y1, x2, topk_idx_out=rec)
    assert torch.equal(plain.forward(y1, x2, topk_idx_out=idx), y2)
    g_off = ((T * k * 4 + 15) // 16) * 16
    s_off = 2 * g_off
    assert torch.equal(rec[: T * k * 4].view(torch.int32).view(T, k), idx)
    gates_fwd = blk.buffer("gates", torch.float32)[: T * k].clone()
    sgate_fwd = blk.buffer("sgate", torch.float32)[:T].clone()
    assert torch.equal(rec[g_off: g_off + T * k * 4].view(torch.float32), gates_fwd)
    assert torch.equal(rec[s_off: s_off + T * 4].view(torch.float32), sgate_fwd)
    # same y1: the record changes nothing
    assert torch.equal(blk.inverse(y1, y2, topk_idx_in=rec), plain.inverse(y1, y2))
    # a y1 that is off by rounding-sized noise: gates still come from the record, bit for bit
    y1p = y1 + 1e-6 * torch.randn_like(y1)
    x2p = blk.inverse(y1p, y2, topk_idx_in=rec)
    assert torch.equal(blk.buffer("gates", torch.float32)[: T * k], gates_fwd)
    assert torch.equal(blk.buffer("sgate", torch.float32)[:T], sgate_fwd)
    assert rel_l2(x2p.cpu().numpy(), s["x2"]) <= TOL_RECON
    x2q = plain.inverse(y1p, y2)          # for comparison: recomputed routing on the perturbed stream
    assert not torch.equal(plain.buffer("gates", torch.float32)[: T * k], gates_fwd)
    assert rel_l2(x2q.cpu().numpy(), s["x2"]) <= TOL_RECON
    # backward through the record equals backward with the remembered indices (same y1: same gates)
    d_a, d_b = torch.zeros_like(y1), torch.zeros_like(y1)
    g_a, g_b = grad_buffers(cfg, w), grad_buffers(cfg, w)
    blk.backward(y1, dy2, d_a, g_a, topk_idx_in=rec)
    plain.backward(y1, dy2, d_b, g_b, topk_idx_in=idx)
    assert blk.status() == 0 and torch.equal(d_a, d_b)
    for n in g_a:
        assert torch.equal(g_a[n], g_b[n]), n
