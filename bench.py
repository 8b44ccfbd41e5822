#!/usr/bin/env python
"""Benchmark of the RevFFN MoE coupling branch on B200.

One step = forward (Eq. 2) + inverse reconstruction + backward by recomputation
of one Qwen1.5-MoE-A2.7B-shaped block over one batch of synthetic tokens
(configuration C1: 8192 tokens).  Prints ONE JSON line.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (independent replicas)
    python bench.py --impl reference        (the CPU oracle on the host cores, bounded sample per step)
    python bench.py --config C3             (24-block reversible stack: tokens/s, peak memory against the
                                             activation-caching variant, reconstruction drift per layer)
    python bench.py --config C4             (token-count sweep 512 .. 65536 on the same block shape)
    python bench.py --config A1             (the attention coupling branch, Eq. 1, of the same block shape)
    python bench.py --config B3             (24 whole RevFFN blocks, both branches: reversible training step,
                                             memory, reconstruction error against fixed-point iterations; B1: one block)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "RevFFN MoE block fwd+inverse+bwd tokens/s; % of B200 bf16 tensor peak"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic per launch (bytes) at C1 from one single-pass ncu capture at full size
# (dram__bytes_read.sum + dram__bytes_write.sum; profiles/tensor_pipe_gemms_C1.md).
# Keyed by pass/kernel; anything else, or any other workload, reports null.
NCU_TRAFFIC_BYTES = {
    "fwd/gemm_expert_gate_up_swiglu": 936_000_000, "inv/gemm_expert_gate_up_swiglu": 1_134_600_000,
    "fwd/gemm_shared_gate_up_swiglu": 185_100_000, "inv/gemm_shared_gate_up_swiglu": 434_600_000,
    "bwd/wgrad_expert_gate_up": 1_660_000_000, "bwd/wgrad_expert_down": 871_600_000,
    "bwd/gemm_expert_du": 1_075_400_000, "bwd/wgrad_shared_gate_up": 425_600_000,
}


NCU_TRAFFIC_SOURCE = ("stored figure, not measured in this run: dram__bytes_read.sum + dram__bytes_write.sum of one "
                      "ncu capture of this kernel at this size, profiles/tensor_pipe_gemms_C1.md")
GROUPED_EXPERT_KERNELS = ("gemm_expert_gate_up_swiglu", "gemm_expert_down_scale", "gemm_expert_dh_dswiglu",
                          "gemm_expert_du", "wgrad_expert_down", "wgrad_expert_gate", "wgrad_expert_up",
                          "wgrad_expert_gate_up")


def pick_tensor_peak(peaks, clocks, timed_s):
    """Which measured bf16 figure a run is held against: the burst figure when the run itself was a burst (a timed
    region under a second, or SM clocks at their maximum while it ran), the sustained one when it ran long enough
    to settle under the power cap.  Returns (key into the peaks, reason)."""
    if not peaks.get("bf16_tflops_sustained"):
        return "bf16_tflops", "no sustained figure available"
    mhz, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    if mhz and mx and mhz >= 0.97 * mx:
        return "bf16_tflops", f"SM clock at its maximum during the run ({mhz:.0f} of {mx:.0f} MHz): burst conditions"
    if timed_s < 1.0:
        return "bf16_tflops", f"timed regions of {timed_s:.2f} s: burst conditions"
    return "bf16_tflops_sustained", (f"{timed_s:.1f} s of timed work at a median SM clock of {mhz:.0f} MHz"
                                     if mhz else f"{timed_s:.1f} s of timed work")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def gemm_flops(cfg, routed_rows):
    """Algorithmic flops per launch of every matrix product, by profiler slot name
    (rows actually routed, not the padded row space)."""
    T, d, h, I, Is = cfg.tokens, cfg.d_model, cfg.h, cfg.d_expert, cfg.d_shared
    R = routed_rows
    return {
        "gemm_p_up": 2 * T * h * d, "gemm_expert_gate_up_swiglu": 2 * R * d * 2 * I,
        "gemm_expert_down_scale": 2 * R * I * d, "gemm_shared_gate_up_swiglu": 2 * T * d * 2 * Is,
        "gemm_shared_down": 2 * T * Is * d, "gemm_p_down_couple": 2 * T * d * h, "gemm_dz": 2 * T * h * d,
        "wgrad_p_down": 2 * T * h * d, "gemm_shared_dh_dswiglu": 2 * T * d * Is, "wgrad_shared_down": 2 * T * d * Is,
        "gemm_shared_du": 2 * T * 2 * Is * d, "wgrad_shared_gate": 2 * T * Is * d, "wgrad_shared_up": 2 * T * Is * d,
        "wgrad_shared_gate_up": 2 * T * 2 * Is * d,
        "gemm_expert_dh_dswiglu": 2 * R * d * I, "gemm_expert_du": 2 * R * 2 * I * d,
        "wgrad_expert_down": 2 * R * d * I, "wgrad_expert_gate": 2 * R * I * d, "wgrad_expert_up": 2 * R * I * d,
        "wgrad_expert_gate_up": 2 * R * 2 * I * d,
        "gemm_dn": 2 * T * d * h, "wgrad_p_up": 2 * T * d * h,
    }


def gemm_bytes(cfg, routed_rows):
    """Algorithmic DRAM bytes per launch of the products whose output is large against their flops (the weight
    gradients of the experts: fp32 [E, I, d]-shaped results from about 546 rows of K each): every operand read
    once, every result written once.  A launch is held against the HBM roofline when these bytes at the measured
    copy bandwidth take longer than its flops at the measured tensor peak."""
    d, I, E = cfg.d_model, cfg.d_expert, cfg.n_experts
    R = routed_rows
    out = E * I * d * 4
    return {"wgrad_expert_down": out + R * d * 2 + R * I * 2, "wgrad_expert_gate": out + R * I * 2 + R * d * 2,
            "wgrad_expert_up": out + R * I * 2 + R * d * 2, "wgrad_expert_gate_up": 2 * out + R * 2 * I * 2 + R * d * 2}


class ClockSampler:
    """nvidia-smi sampling of SM clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.strip().split(", ") for r in open(self.tmp.name).read().strip().splitlines() if r.strip()]
        os.unlink(self.tmp.name)
        clocks, power, reasons, mx = [], [], set(), None
        for r in rows:
            if len(r) < 9:
                continue
            try:
                clocks.append(float(r[1])); mx = float(r[2]); power.append(float(r[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if clocks:
            # under load = samples drawing real power (idle samples at the edges are dropped)
            busy = [c for c, p in zip(clocks, power) if p >= 0.5 * max(power)] or clocks
            out.update(sm_mhz=float(np.median(busy)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(clocks),
                       power_w_max=max(power))
        return out


def oracle_step(orc, w, s, cfg, n_tok):
    """forward + inverse + backward of the oracle on the first n_tok tokens."""
    y1, x2, dy2 = s["y1"][:n_tok], s["x2"][:n_tok], s["dy2"][:n_tok]
    y2, _ = orc.forward(w, y1, x2, cfg.top_k, cfg.norm_eps)
    orc.inverse(w, y1, y2, cfg.top_k, cfg.norm_eps)
    orc.backward(w, y1, dy2, cfg.top_k, cfg.norm_eps)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    """The CPU oracle, as it stands, on the host cores; each step a bounded token sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import revffn_oracle as orc
    from workloads import make_streams, make_weights
    w = make_weights(cfg, args.seed)
    s = make_streams(cfg, args.seed)
    # the sample shrinks until the whole run (warm-up + timed steps) fits a few minutes on this host;
    # most of a small step is widening the weights of the experts its tokens reach, so fewer tokens help
    n_tok = args.cpu_sample_tokens
    budget_s = 150.0
    while True:
        t0 = time.perf_counter()
        oracle_step(orc, w, s, cfg, n_tok)
        if (time.perf_counter() - t0) * (args.steps + args.warmup) <= budget_s or n_tok <= 4:
            break
        n_tok = max(4, n_tok // 2)
    for _ in range(args.warmup):
        oracle_step(orc, w, s, cfg, n_tok)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(orc, w, s, cfg, n_tok)
    dt = time.perf_counter() - t0
    value = n_tok * args.steps / dt
    cores = blas_threads()
    sample = f"first {n_tok} of {cfg.tokens} tokens per step, full weights, fp64 numpy"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.tokens} tokens, d={cfg.d_model}, E={cfg.n_experts}, k={cfg.top_k}, "
                               f"I={cfg.d_expert}, I_s={cfg.d_shared}", "sample_tokens": n_tok},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(values, world, device="cuda"):
    """Element-wise maximum of a list of floats over all ranks (the slowest replica sets the job's time)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_tokens_per_s(world, tokens_per_rank, steps, ms_total):
    """Whole-job throughput of `world` independent replicas that each ran `steps` steps in ms_total."""
    return world * tokens_per_rank * steps / (ms_total * 1e-3)


def replica_seed(seed, rank):
    """Every replica draws its own tokens; the weights are the same on all of them."""
    return seed + rank


def dist_setup():
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1 and not dist.is_initialized():
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
    return rank, world, local, barrier


def run_ours(args, cfg):
    out = measure_block(args, cfg, e2e=not args.steps_only, cpu=not (args.no_cpu_baseline or args.steps_only),
                        steps_only=args.steps_only)
    if out is not None:
        print(json.dumps(out))
    finish()


def finish():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def measure_block(args, cfg, e2e=True, cpu=True, w_dev=None, w_host=None, steps_only=False):
    """One block at cfg.tokens tokens per GPU; returns the JSON record (rank 0) or None."""
    import torch
    import torch.distributed as dist
    import paper_2512_20920_b200 as rv
    from workloads import make_streams, make_weights

    rank, world, local, barrier = dist_setup()

    # every rank is an independent replica with its own tokens (seed + rank); weights are the same
    if w_dev is None:
        w_host = make_weights(cfg, args.seed)
        wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
        w_dev = {n: torch.from_numpy(v).cuda().to(torch.float32 if n in ("norm_gamma", "b_router") else wdt).contiguous()
                 for n, v in w_host.items()}
    s_host = make_streams(cfg, replica_seed(args.seed, rank))
    blk = rv.Block(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k,
                   d_expert=cfg.d_expert, d_shared=cfg.d_shared,
                   weight_dtype=rv.BF16 if cfg.weight_dtype == "bf16" else rv.F32, weights=w_dev,
                   norm_eps=cfg.norm_eps, flags=rv.FLAG_GATE_SOFTMAX_ALL if args.gating == "softmax_all" else 0)
    y1, x2, dy2 = (torch.from_numpy(s_host[n]).cuda() for n in ("y1", "x2", "dy2"))
    y2, x2r, dy1 = torch.empty_like(x2), torch.empty_like(x2), torch.zeros_like(y1)
    # routers stay frozen (Sec. 3.3 of the paper); every other weight gets its fp32 gradient
    grads = {n: torch.empty(v.shape, dtype=torch.float32, device="cuda") for n, v in w_dev.items()
             if n not in ("w_router", "b_router")}

    def step():
        # Inverse and gradient pass share one evaluation of the branch (the gradient pass of a reversible
        # block needs exactly the intermediates the inverse pass has just recomputed).
        # The weights do not change between the passes of a step, so the router folded through P_up by the
        # forward pass is still valid when the inverse pass starts (REVFFN_FLAG_ROUTER_FOLDED).
        blk.forward(y1, x2, y2)
        blk.inverse(y1, y2, x2r, save=True, flags=rv.FLAG_ROUTER_FOLDED)
        blk.backward(y1, dy2, dy1, grads, reuse=True)

    def step_single():
        # the same step with every launch on one stream (the library's second stream switched off)
        blk.forward(y1, x2, y2, flags=rv.FLAG_SINGLE_STREAM)
        blk.inverse(y1, y2, x2r, save=True, flags=rv.FLAG_ROUTER_FOLDED | rv.FLAG_SINGLE_STREAM)
        blk.backward(y1, dy2, dy1, grads, reuse=True, flags=rv.FLAG_SINGLE_STREAM)

    def step_unshared():
        # every pass recomputes the branch on its own
        blk.forward(y1, x2, y2)
        blk.inverse(y1, y2, x2r)
        blk.backward(y1, dy2, dy1, grads)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert blk.status() == 0, "device status word set during warm-up"
    routed_rows = cfg.tokens * cfg.top_k

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    # timed region: K steps, CUDA events on the launching stream, no per-launch instrumentation
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = rv.revffn_prof_launches()
    barrier()
    if sampler:
        sampler.start()
    ms_total = timed(step, args.steps)
    clocks = sampler.stop() if sampler else None
    launches = rv.revffn_prof_launches() - launches0
    assert blk.status() == 0, "device status word set during the timed region"
    if steps_only:
        ms_total = max_over_ranks([ms_total], world)[0]
        if rank != 0:
            return None
        return {"metric": METRIC, "value": job_tokens_per_s(world, cfg.tokens, args.steps, ms_total), "unit": "tokens/s",
                "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"{cfg.name}: steps only"}, "gpu_launches": int(launches), "clocks": clocks}
    # the same K steps again with an event pair around every launch: per-kernel durations
    rv.revffn_prof_enable(True)
    barrier()
    sampler2 = ClockSampler(local) if rank == 0 else None
    if sampler2:
        sampler2.start()
    ms_prof_total = timed(step, args.steps)
    clocks_prof = sampler2.stop() if sampler2 else None
    if clocks_prof and not clocks_prof.get("sm_mhz"):
        clocks_prof = None
    prof = rv.revffn_prof_collect()
    rv.revffn_prof_enable(False)
    # and the variant in which no pass shares anything (short)
    n_un = max(3, min(args.steps, 20))
    step_unshared()
    barrier()
    ms_unshared = timed(step_unshared, n_un) / n_un
    step_single()
    barrier()
    ms_single = timed(step_single, n_un) / n_un
    # the FP8 variant of the routed experts (forward and inverse passes only): same block, e4m3 expert operands
    fp8_rec = None
    if cfg.weight_dtype == "bf16" and cfg.d_model <= 2048 and cfg.d_model % 256 == 0 and args.gating == "renorm":
        blk8 = rv.Block(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k,
                        d_expert=cfg.d_expert, d_shared=cfg.d_shared, weight_dtype=rv.BF16, weights=w_dev,
                        norm_eps=cfg.norm_eps, flags=rv.FLAG_FP8_EXPERTS, workspace=blk.ws, backward=False)
        blk8.quantize_experts()

        def fwd_inv(b):
            b.forward(y1, x2, y2)
            b.inverse(y1, y2, x2r, flags=rv.FLAG_ROUTER_FOLDED)

        n8 = max(3, min(args.steps, 20))
        for b in (blk8, blk):
            fwd_inv(b)
        barrier()
        ms8 = timed(lambda: fwd_inv(blk8), n8) / n8
        ms16 = timed(lambda: fwd_inv(blk), n8) / n8
        rv.revffn_prof_enable(True)
        fwd_inv(blk8)
        torch.cuda.synchronize()
        p8 = rv.revffn_prof_collect()
        rv.revffn_prof_enable(False)
        assert blk8.status() == 0
        f8_flops = gemm_flops(cfg, routed_rows)
        fp8_rec = {"fwd_plus_inv_ms": ms8, "bf16_fwd_plus_inv_ms": ms16,
                   "expert_gate_up_ms": p8.get("fwd/gemm_expert_gate_up_swiglu", (0, 0))[0],
                   "expert_gate_up_tflops": f8_flops["gemm_expert_gate_up_swiglu"] / max(p8.get("fwd/gemm_expert_gate_up_swiglu", (1e9, 0))[0], 1e-9) / 1e9,
                   "expert_down_ms": p8.get("fwd/gemm_expert_down_scale", (0, 0))[0],
                   "expert_down_tflops": f8_flops["gemm_expert_down_scale"] / max(p8.get("fwd/gemm_expert_down_scale", (1e9, 0))[0], 1e-9) / 1e9,
                   "gather_and_quantise_ms": p8.get("fwd/gather_u", (0, 0))[0],
                   "note": "routed experts' three products on e4m3 operands with per-row scales (REVFFN_FLAG_FP8_EXPERTS); "
                           "branch output about 4-5 % (relative L2) from the bf16 evaluation; not part of the headline"}
        del blk8
    ms_total, ms_unshared, ms_single = max_over_ranks([ms_total, ms_unshared, ms_single], world)
    ms_step = ms_total / args.steps
    ms_prof_step = ms_prof_total / args.steps
    value = job_tokens_per_s(world, cfg.tokens, args.steps, ms_total)

    e2e_value, e2e_sync_value, dt, dt_sync, bytes_dir = None, None, 0.0, 0.0, 0
    if e2e:
        # end to end: host-resident streams, H2D and D2H copies inside the timed region
        pin = lambda a: torch.from_numpy(a).pin_memory()
        hy1, hx2, hdy2 = pin(s_host["y1"]), pin(s_host["x2"]), pin(s_host["dy2"])
        hy2, hx2r, hdy1 = (torch.empty_like(hy1).pin_memory() for _ in range(3))
        slot = ((hy1.numel() * 4 + 255) // 256) * 256
        staging = torch.empty(12 * slot, dtype=torch.uint8, device="cuda")
        g_struct = blk.grads_struct(grads)
        copy_stream = torch.cuda.Stream()
        # (1) one step at a time: the host waits for a step's results before it starts the next one
        host_step = lambda: rv.revffn_moe_step_host(blk.desc, blk.w, g_struct, hy1, hx2, hdy2, hy2, hx2r, hdy1, staging,
                                                    blk.ws, copy_stream=copy_stream.cuda_stream)
        for _ in range(2):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            host_step()
            torch.cuda.synchronize()     # the step's results are read on the host
        dt_sync = time.perf_counter() - t0
        dt_sync = max_over_ranks([dt_sync], world)[0]
        # (2) a loop of steps, pipelined: every step still uploads its inputs from pinned host memory and
        # downloads its results, and the host waits for the results of step i - 1 while step i runs; the
        # transfers of neighbouring steps run beside the passes (two staging sets, two sets of host outputs)
        outs = [(hy2, hx2r, hdy1), tuple(torch.empty_like(hy1).pin_memory() for _ in range(3))]
        def piped(n_steps):
            prev = None
            for i in range(n_steps):
                o = outs[i & 1]
                rv.revffn_moe_step_host(blk.desc, blk.w, g_struct, hy1, hx2, hdy2, o[0], o[1], o[2], staging, blk.ws,
                                        copy_stream=copy_stream.cuda_stream, pipelined=True)
                ev = torch.cuda.Event()
                ev.record(copy_stream)
                if prev is not None:
                    prev.synchronize()   # the previous step's results are on the host
                prev = ev
            prev.synchronize()
            torch.cuda.synchronize()
        piped(3)
        barrier()
        t0 = time.perf_counter()
        piped(args.steps)
        dt = time.perf_counter() - t0
        dt = max_over_ranks([dt], world)[0]
        e2e_value = job_tokens_per_s(world, cfg.tokens, args.steps, dt * 1e3)
        e2e_sync_value = job_tokens_per_s(world, cfg.tokens, args.steps, dt_sync * 1e3)
        bytes_dir = 3 * hy1.numel() * 4

    # the optimiser step fused into the weight-gradient products (last: it changes the weights, by steps far below
    # their last bit): inverse + backward with the gradients written, with the fused SGD step, with the fused Adam step
    fused_rec = None
    peak_device_bytes = int(torch.cuda.max_memory_allocated())      # before the moment buffers of the Adam leg
    if e2e and cfg.weight_dtype == "bf16" and args.gating == "renorm":
        names = [n for n in rv.UPD_NAMES if n in blk.weights]
        rest = {n: t for n, t in grads.items() if n not in names}
        mom = {n: torch.zeros_like(blk.weights[n], dtype=torch.float32) for n in names}
        var = {n: torch.zeros_like(blk.weights[n], dtype=torch.float32) for n in names}
        adam_t = [0]

        def inv_bwd(upd):
            blk.inverse(y1, y2, x2r, save=True)
            if upd == "adam":
                adam_t[0] += 1
                blk.backward(y1, dy2, dy1, rest, reuse=True, sgd=rv.make_adam(1e-9, adam_t[0], names, mom, var))
            elif upd == "sgd":
                blk.backward(y1, dy2, dy1, rest, reuse=True, sgd=rv.make_sgd(1e-9, names))
            else:
                blk.backward(y1, dy2, dy1, grads, reuse=True)

        n_f = max(3, min(args.steps, 10))
        fused_ms = {}
        for upd in ("none", "sgd", "adam"):
            inv_bwd(upd)
            barrier()
            fused_ms[upd] = timed(lambda: inv_bwd(upd), n_f) / n_f
        assert blk.status() == 0
        fused_rec = {"inverse_plus_backward_ms": {"gradients_written": fused_ms["none"], "fused_sgd": fused_ms["sgd"],
                                                  "fused_adam": fused_ms["adam"]},
                     "gradient_bytes_not_written": int(sum(blk.weights[n].numel() for n in names) * 4),
                     "note": "revffn_moe_backward_sgd / revffn_moe_backward_adam with all eight matrices in the mask; "
                             "not part of the headline step"}
        del mom, var

    if rank != 0:
        return None

    peaks, peak_kind = load_peaks()
    flops = gemm_flops(cfg, routed_rows)
    # per-pass and per-kernel accounting
    passes = {"fwd": 0.0, "inv": 0.0, "bwd": 0.0}
    kernels = []
    # A profiler slot is one product (or kernel) of one pass; some products run as several launches (row pairs +
    # odd tiles of the experts, K slices + their sum): the slot's time is the sum, its flops are counted once per
    # step.  `cnt` below is therefore the number of times the PRODUCT ran (= steps), `launches` the kernel launches.
    slot_launches = {}
    for name, (ms, launches_) in prof.items():
        ps, kn = name.split("/")
        passes[ps] += ms / args.steps
        slot_launches[name] = launches_
        kernels.append((ms, args.steps, name, kn))
    kernels.sort(reverse=True)
    step_flops = {"fwd": 0.0, "inv": 0.0, "bwd": 0.0}
    for ms, cnt, name, kn in kernels:
        if kn in flops:
            step_flops[name.split("/")[0]] += flops[kn] * cnt / args.steps
    total_flops = sum(step_flops.values())
    # dominant kernel = the matrix product with the largest share of the step
    dom = next(((ms, cnt, name, kn) for ms, cnt, name, kn in kernels if kn in flops), None)
    peak_name, peak_why = pick_tensor_peak(peaks, clocks_prof or clocks, 1e-3 * ms_total)
    peak = peaks[peak_name]
    burst, sustained = peaks["bf16_tflops"], peaks.get("bf16_tflops_sustained")
    sm_mhz = (clocks_prof or clocks or {}).get("sm_mhz")
    n_sms = torch.cuda.get_device_properties(local).multi_processor_count

    def tensor_fractions(tflops):
        """The same figure against both measured denominators and, clock-normalised, in dense bf16 flop per SM
        clock (nominal 8192 per SM and clock), so that runs at different SM clocks can be compared."""
        rec = {"tflops": tflops, "frac_burst": tflops / burst, "frac_sustained": tflops / sustained if sustained else None}
        if sm_mhz:
            per_clk = tflops * 1e12 / (sm_mhz * 1e6 * n_sms)
            rec.update(flop_per_sm_clk=per_clk, frac_of_8192_per_sm_clk=per_clk / 8192.0, sm_mhz=sm_mhz)
        return rec

    roofline = None
    grouped = [k for k in kernels if k[3] in GROUPED_EXPERT_KERNELS]
    g_fl = sum(flops[k[3]] * k[1] for k in grouped)
    g_ms = sum(k[0] for k in grouped)
    if dom:
        ms, cnt, name, kn = dom
        achieved = flops[kn] / (ms / cnt * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": name, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": achieved / peak,
                    "peak_source": f"{peak_kind}: {peak_name} of MEASURED_PEAKS.json ({peak_why})",
                    "dominant": tensor_fractions(achieved),
                    "traffic": NCU_TRAFFIC_BYTES.get(name) if cfg.name == "C1" else None,
                    "traffic_source": NCU_TRAFFIC_SOURCE if (cfg.name == "C1" and name in NCU_TRAFFIC_BYTES) else None,
                    "launch_ms": ms / cnt,
                    "share_of_step": ms / (ms_prof_step * args.steps),
                    "timed_over": f"a second pass of the same {args.steps} steps with a CUDA-event pair around "
                                  f"every launch ({ms_prof_step:.3f} ms per step against {ms_step:.3f} without)"}
        nbytes = gemm_bytes(cfg, routed_rows).get(kn)
        if nbytes and nbytes / (peaks["hbm_gbs"] * 1e9) > flops[kn] / (peak * 1e12):
            # this launch moves more bytes than it can compute on: HBM is its roofline
            gbs = nbytes / (ms / cnt * 1e-3) / 1e9
            roofline.update(bound="hbm", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s", frac=gbs / peaks["hbm_gbs"],
                            peak_source=f"{peak_kind}: hbm_gbs of MEASURED_PEAKS.json (copy bandwidth)",
                            algorithmic_bytes=nbytes, traffic=NCU_TRAFFIC_BYTES.get(name) if cfg.name == "C1" else None,
                            traffic_source=NCU_TRAFFIC_SOURCE if (cfg.name == "C1" and name in NCU_TRAFFIC_BYTES) else None,
                            why=f"{nbytes / 1e6:.0f} MB of operands and fp32 results at the copy bandwidth take "
                                f"{nbytes / (peaks['hbm_gbs'] * 1e9) * 1e3:.3f} ms, its {flops[kn] / 1e12:.3f} TFLOP at the tensor peak "
                                f"{flops[kn] / (peak * 1e12) * 1e3:.3f} ms; the tensor view of the same launch is under 'dominant'")
        # the largest launch that the tensor pipe bounds, for comparison with earlier records
        dom_t = next(((m_, c_, n_, k_) for m_, c_, n_, k_ in kernels if k_ in flops and k_ not in gemm_bytes(cfg, routed_rows)), None)
        if dom_t:
            roofline["largest_tensor_bound_launch"] = dict(tensor_fractions(flops[dom_t[3]] / (dom_t[0] / dom_t[1] * 1e-3) / 1e12),
                                                           kernel=dom_t[2], launch_ms=dom_t[0] / dom_t[1],
                                                           traffic=NCU_TRAFFIC_BYTES.get(dom_t[2]) if cfg.name == "C1" else None)
        if g_ms > 0:
            # the quantity the target is stated on: every expert-grouped product of the step together
            roofline["grouped"] = dict(tensor_fractions(g_fl / (g_ms * 1e-3) / 1e12), ms_per_step=g_ms / args.steps,
                                       launches_per_step=sum(slot_launches[k[2]] for k in grouped) / args.steps,
                                       share_of_step=g_ms / (ms_prof_step * args.steps),
                                       kernels=sorted({k[3] for k in grouped}))
        roofline["whole_step"] = tensor_fractions(total_flops / (ms_step * 1e-3) / 1e12)
    top = [{"kernel": name, "ms_per_step": ms / args.steps, "launches_per_step": slot_launches[name] / args.steps,
            "tflops": (flops[kn] * cnt / (ms * 1e-3) / 1e12) if kn in flops and ms > 0 else None}
           for ms, cnt, name, kn in kernels]

    # CPU baseline: the oracle as it stands on a bounded sample of the same workload (rank 0, N = 1 only)
    cpu_rec = None
    if world == 1 and cpu and w_host is not None:
        from oracle import revffn_oracle as orc
        n_tok = args.cpu_sample_tokens
        oracle_step(orc, w_host, s_host, cfg, n_tok)      # first call pays for first-touch of its gradient arrays
        t0 = time.perf_counter()
        oracle_step(orc, w_host, s_host, cfg, n_tok)
        cdt = time.perf_counter() - t0
        cpu_rec = {"value": n_tok / cdt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
               "sample": f"second of two fwd+inverse+bwd passes over the first {n_tok} of {cfg.tokens} tokens, "
                         f"full weights, fp64 numpy, {cdt:.1f} s; most of that time widens the 1.1 GB of bf16-valued "
                         f"weights to fp64 on every call, which the oracle does by design"}

    peak_t = peak
    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: one Qwen1.5-MoE-A2.7B-shaped block, {cfg.tokens} tokens per GPU, "
                               f"d={cfg.d_model}, E={cfg.n_experts}, top-{cfg.top_k}, I={cfg.d_expert}, "
                               f"I_s={cfg.d_shared}; step = forward + inverse + backward (all weight gradients "
                               f"in fp32 except the frozen router); the backward pass reuses the branch "
                               f"evaluation of the inverse pass, the inverse pass the folded router of the forward pass" + ("; gates not renormalised" if args.gating != "renorm" else ""),
                   "l2": "per-step working set (1.1 GB weights + >2 GB activations) exceeds the 126 MB L2",
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "pct_bf16_tensor_peak": 100.0 * total_flops / (ms_step * 1e-3) / 1e12 / peak_t,
        "step_tflops": total_flops / (ms_step * 1e-3) / 1e12,
        "unshared": {"ms_per_step": ms_unshared, "value": world * cfg.tokens / (ms_unshared * 1e-3),
                     "note": "forward, inverse and backward each recompute the branch (3 evaluations, not 2)"},
        "single_stream": {"ms_per_step": ms_single, "value": world * cfg.tokens / (ms_single * 1e-3),
                          "note": "REVFFN_FLAG_SINGLE_STREAM: the shared expert and the weight gradients queue behind "
                                  "the other launches instead of running beside them on the library's second stream; "
                                  "the per-kernel figures (profiler on) are taken in this form"},
        "passes_ms": passes,
        "passes_tokens_per_s": {k: (cfg.tokens / (v * 1e-3) if v > 0 else None) for k, v in passes.items()},
        "grouped_expert_gemms": {"tflops": g_fl / (g_ms * 1e-3) / 1e12 if g_ms > 0 else None,
                                 "frac_of_peak": (g_fl / (g_ms * 1e-3) / 1e12 / peak_t) if g_ms > 0 else None,
                                 "peak": peak_name, "ms_per_step": g_ms / args.steps},
        "kernels": top,
        "fp8_experts": fp8_rec,
        "fused_update": fused_rec,
        "roofline": roofline,
        "cpu_baseline": cpu_rec,
        "e2e": ({"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": bytes_dir,
                 "d2h_bytes_per_step": bytes_dir, "ms_per_step": 1e3 * dt / args.steps,
                 "mode": "loop of revffn_moe_step_host calls in the pipelined form: each step uploads its three "
                         "input streams from pinned host memory and downloads its three result streams; the host "
                         "waits for the results of step i-1 while step i runs",
                 "one_step_at_a_time": {"value": e2e_sync_value, "ms_per_step": 1e3 * dt_sync / args.steps,
                                        "note": "host synchronises after every step before starting the next"}}
                if e2e else None),
        "gpu_launches": int(launches),
        "clocks": clocks,
        "clocks_per_kernel_pass": clocks_prof,
        "peak_device_bytes": peak_device_bytes,
        "workspace_bytes": {"fwd": blk.fwd_bytes, "bwd": blk.bwd_bytes},
    }
    # achieved GB/s of the copy-like kernels (algorithmic bytes: rows read + rows written)
    T, d, k_ = cfg.tokens, cfg.d_model, cfg.top_k
    hbm_bytes = {"gather_u": 2 * routed_rows * d * 2, "gather_dz": 2 * routed_rows * d * 2,
                 "combine": (k_ + 2) * T * d * 2, "du_reduce": (k_ + 2) * T * d * 2}
    out["hbm_kernels"] = {name: {"gbs": hbm_bytes[kn] * cnt / (ms * 1e-3) / 1e9,
                                 "frac_of_peak": hbm_bytes[kn] * cnt / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                          for ms, cnt, name, kn in kernels if kn in hbm_bytes and ms > 0}
    return out


def run_sweep(args):
    """C4: the C1 block shape at 512 .. 65536 tokens; one record per size in one JSON line."""
    import torch
    from workloads import CONFIGS, make_weights
    rank, world, local, barrier = dist_setup()
    base = CONFIGS["C1"]
    w_host = make_weights(base, args.seed)
    w_dev = {n: torch.from_numpy(v).cuda().to(torch.float32 if n in ("norm_gamma", "b_router") else torch.bfloat16)
             .contiguous() for n, v in w_host.items()}
    del w_host
    recs = []
    for t in (512, 2048, 8192, 32768, 65536):
        cfg = CONFIGS[f"C4-{t}"]
        a = argparse.Namespace(**vars(args))
        a.steps = max(5, min(args.steps, int(args.steps * 8192 / t)))      # about the same timed work per size
        r = measure_block(a, cfg, e2e=False, cpu=False, w_dev=w_dev)
        torch.cuda.empty_cache()
        if r is None:
            continue
        bwd_gemm = [k for k in r["kernels"] if k["tflops"]]
        recs.append({"tokens": t, "steps": a.steps, "ms_per_step": r["ms_per_step"], "tokens_per_s": r["value"],
                     "passes_tokens_per_s": r["passes_tokens_per_s"], "step_tflops": r["step_tflops"],
                     "pct_bf16_tensor_peak": r["pct_bf16_tensor_peak"],
                     "grouped_expert_gemms_frac_of_peak": r["grouped_expert_gemms"]["frac_of_peak"],
                     "hbm_kernels": r["hbm_kernels"], "clocks": r["clocks"],
                     "slowest_gemm": min(bwd_gemm, key=lambda k: k["tflops"])["kernel"] if bwd_gemm else None})
    if rank == 0:
        mid = next(x for x in recs if x["tokens"] == 8192)
        peaks, kind = load_peaks()
        print(json.dumps({
            "metric": METRIC, "value": mid["tokens_per_s"], "unit": "tokens/s", "n_gpus": world, "steps": mid["steps"],
            "warmup": max(args.warmup, 3), "ms_per_step": mid["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C4: token-count sweep on the C1 block shape; value is the 8192-token point",
                       "l2": "working set exceeds the 126 MB L2 at every size (1.1 GB of weights per pass)"},
            "peak": {"bf16_tflops_sustained": peaks.get("bf16_tflops_sustained"), "hbm_gbs": peaks.get("hbm_gbs"),
                     "source": kind},
            "sweep": recs}))
    finish()


def run_stack(args, cfg):
    """C3: n_blocks coupling branches; step = forward through the stack + reversible backward."""
    import torch
    import paper_2512_20920_b200 as rv
    from workloads import make_streams, make_weights_device, weight_shapes
    rank, world, local, barrier = dist_setup()
    L = args.blocks or cfg.n_blocks
    weights = [make_weights_device(cfg, args.seed, block=l) for l in range(L)]
    w_bytes = sum(t.numel() * t.element_size() for w in weights for t in w.values())
    s_host = make_streams(cfg, replica_seed(args.seed, rank))
    a0, b0 = torch.from_numpy(s_host["y1"]).cuda(), torch.from_numpy(s_host["x2"]).cuda()
    g0 = torch.from_numpy(s_host["dy2"]).cuda()
    # one fp32 gradient buffer per tensor, reused by every layer (an optimiser would consume it layer by layer);
    # the router stays frozen
    gbuf = {n: torch.empty(shp, dtype=torch.float32, device="cuda") for n, shp in weight_shapes(cfg).items()
            if n not in ("w_router", "b_router")}
    a, b, ga, gb = (torch.empty_like(a0) for _ in range(4))
    kw = dict(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k, d_expert=cfg.d_expert,
              d_shared=cfg.d_shared, weight_dtype=rv.BF16, weights=weights, norm_eps=cfg.norm_eps)

    def timed_variant(caching, records=False):
        torch.cuda.synchronize()
        base_alloc = torch.cuda.memory_allocated()
        torch.cuda.reset_peak_memory_stats()
        stk = rv.Stack(caching=caching, flags=rv.FLAG_ROUTING_RECORD if records else 0, **kw)
        garr = stk.grads_array([gbuf] * L)
        # routing records: forward remembers every layer's expert sets and gate values, backward runs no router
        routing = torch.empty(L * stk.record_bytes, dtype=torch.uint8, device="cuda") if records else None

        def step():
            a.copy_(a0); b.copy_(b0); ga.copy_(g0); gb.copy_(g0)
            stk.forward(a, b, routing)
            stk.backward(a, b, ga, gb, garr, topk_idx=routing)

        for _ in range(max(args.warmup, 3)):
            step()
        torch.cuda.synchronize()
        assert stk.status() == 0
        l0 = rv.revffn_prof_launches()
        barrier()
        sampler = ClockSampler(local) if rank == 0 else None
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        clocks = sampler.stop() if sampler else None
        ms = max_over_ranks([e0.elapsed_time(e1)], world)[0] / args.steps
        assert stk.status() == 0
        rec = {"ms_per_step": ms, "tokens_per_s": cfg.tokens / (ms * 1e-3), "launches": rv.revffn_prof_launches() - l0,
               "activation_bytes": int(torch.cuda.max_memory_allocated() - base_alloc),
               "peak_device_bytes": int(torch.cuda.max_memory_allocated()), "clocks": clocks,
               "workspace_bytes": stk.bwd_bytes, "cache_bytes": 0 if stk.cache is None else stk.cache.numel(),
               "saved_bytes_per_layer": stk.saved_bytes}
        rec["recon_rel_l2"] = [float((a - a0).norm() / a0.norm()), float((b - b0).norm() / b0.norm())] if not caching else None
        del stk, garr
        torch.cuda.empty_cache()
        return rec

    rev = timed_variant(False)
    rec = timed_variant(False, records=True)
    cac = timed_variant(True)

    # reconstruction drift and routing flips per layer (diagnostic pass, not timed): layer by layer through
    # the single-layer entry points, keeping every layer's streams and expert sets from the forward sweep
    drift = None
    if not args.no_drift and rank == 0:
        mk = lambda w, ws: rv.Block(tokens=cfg.tokens, d_model=cfg.d_model, n_experts=cfg.n_experts, top_k=cfg.top_k,
                                    d_expert=cfg.d_expert, d_shared=cfg.d_shared, weight_dtype=rv.BF16, weights=w,
                                    norm_eps=cfg.norm_eps, workspace=ws, backward=False)
        first = mk(weights[0], None)
        blks = [first] + [mk(w, first.ws) for w in weights[1:]]      # one workspace for all layers
        drift = {}
        for mode in ("recomputed_routing", "remembered_routing"):
            s = [a0.clone(), b0.clone()]
            kept, idxs = [], []
            for l, blk in enumerate(blks):
                P, R = (s[0], s[1]) if l % 2 == 0 else (s[1], s[0])
                kept.append(R.clone())
                idx = torch.empty(cfg.tokens, cfg.top_k, dtype=torch.int32, device="cuda")
                blk.forward(P, R, R, topk_idx_out=idx)
                idxs.append(idx)
            per_layer = []
            for l in reversed(range(L)):
                blk = blks[l]
                P, R = (s[0], s[1]) if l % 2 == 0 else (s[1], s[0])
                blk.inverse(P, R, R, topk_idx_in=idxs[l] if mode == "remembered_routing" else None)
                idx_now = blk.buffer("idx", torch.int32)[: cfg.tokens * cfg.top_k].view(cfg.tokens, cfg.top_k)
                flips = int((idx_now.sort(dim=1).values != idxs[l].sort(dim=1).values).any(dim=1).sum())
                per_layer.append({"layer": l, "rel_l2": float((R - kept[l]).norm() / kept[l].norm()),
                                  "max_abs": float((R - kept[l]).abs().max()), "routing_flips": flips})
            drift[mode] = per_layer[::-1]
        del blks, kept, idxs

    if rank != 0:
        finish()
        return
    print(json.dumps({
        "metric": METRIC, "value": world * rev["tokens_per_s"], "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": rev["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"C3: {L}-block reversible stack of the C1 block, {cfg.tokens} tokens per GPU; step = "
                               f"forward through all layers + backward by layer-wise inverse reconstruction (no "
                               f"cached activations); streams swap roles between layers (only the MoE branch of "
                               f"each block exists here); weights drawn on the device",
                   "l2": "per-layer working set exceeds the 126 MB L2", "blocks": L},
        "gpu_launches": int(rev["launches"]), "clocks": rev["clocks"],
        "reversible": rev, "reversible_with_routing_records": rec, "caching": cac,
        "memory": {"weights_bytes": w_bytes,
                   "reversible_activation_bytes": rev["activation_bytes"],
                   "caching_activation_bytes": cac["activation_bytes"],
                   "caching_saved_bytes_minimum": L * (cac["saved_bytes_per_layer"] + a0.numel() * 4),
                   "note": "activation bytes = peak allocation above weights, streams and the shared gradient "
                           "buffers while the variant ran; the caching variant allocates a full workspace per "
                           "layer, of which saved_bytes_per_layer (+ the layer's input stream) must be kept"},
        "speed_ratio_reversible_over_caching": cac["ms_per_step"] / rev["ms_per_step"],
        "drift": drift}))
    finish()


def run_block_stack(args, acfg, mcfg, layers):
    """B3 / B1: a stack of whole RevFFN blocks (Eq. 1 then Eq. 2 per block); step = forward through all layers +
    reversible back-propagation (every layer's inputs rebuilt from its outputs, nothing cached)."""
    import torch
    import paper_2512_20920_b200 as rv
    from workloads import make_weights_device, weight_shapes
    from workloads.generate import attn_weight_shapes, make_attn_streams, make_attn_weights_device
    rank, world, local, barrier = dist_setup()
    L = args.blocks or layers
    wm = [make_weights_device(mcfg, args.seed, block=l) for l in range(L)]
    wa = [make_attn_weights_device(acfg, args.seed, block=l) for l in range(L)]
    w_bytes = sum(t.numel() * t.element_size() for ws in (wm, wa) for w in ws for t in w.values())
    s_host = make_attn_streams(acfg, replica_seed(args.seed, rank))
    x1, x2, d1, d2 = (torch.from_numpy(s_host[n]).cuda() for n in ("x1", "x2", "dy1", "dx2"))
    # one fp32 gradient buffer per tensor, reused by every layer; the router stays frozen (Sec. 3.3)
    gm_buf = {n: torch.empty(shp, dtype=torch.float32, device="cuda") for n, shp in weight_shapes(mcfg).items()
              if n not in ("w_router", "b_router")}
    ga_buf = {n: torch.empty(shp, dtype=torch.float32, device="cuda") for n, shp in attn_weight_shapes(acfg).items()}
    torch.cuda.synchronize()
    base_alloc = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    stk = rv.RevStack(batch=acfg.batch, seq_len=acfg.seq_len, d_model=acfg.d_model, n_heads=acfg.n_heads,
                      n_kv_heads=acfg.n_kv_heads, n_experts=mcfg.n_experts, top_k=mcfg.top_k, d_expert=mcfg.d_expert,
                      d_shared=mcfg.d_shared, weight_dtype=rv.BF16, attn_weights=wa, moe_weights=wm, inverse_iters=1,
                      norm_eps=mcfg.norm_eps, rope_theta=acfg.rope_theta)
    ga, gm = stk.grads_arrays([ga_buf] * L, [gm_buf] * L)
    a, b, g1, g2 = (torch.empty_like(x1) for _ in range(4))
    idx = torch.empty(L, acfg.tokens, mcfg.top_k, dtype=torch.int32, device="cuda")

    def step(iters=None, remember=False):
        a.copy_(x1); b.copy_(x2); g1.copy_(d1); g2.copy_(d2)
        stk.forward(a, b, idx if remember else None)
        stk.backward(a, b, g1, g2, ga, gm, topk_idx=idx if remember else None, inverse_iters=iters)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert stk.status() == 0
    l0 = rv.revffn_prof_launches()
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    if sampler:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    ms = max_over_ranks([e0.elapsed_time(e1)], world)[0] / args.steps
    launches = rv.revffn_prof_launches() - l0
    assert stk.status() == 0
    act_bytes = int(torch.cuda.max_memory_allocated() - base_alloc)

    # per-pass split (one step with an event pair around each sweep)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    a.copy_(x1); b.copy_(x2); g1.copy_(d1); g2.copy_(d2)
    ev[0].record(); stk.forward(a, b, None); ev[1].record(); stk.backward(a, b, g1, g2, ga, gm); ev[2].record()
    torch.cuda.synchronize()
    split = {"forward_ms": ev[0].elapsed_time(ev[1]), "backward_ms": ev[1].elapsed_time(ev[2])}

    # reconstruction error of the stack's inputs after the backward sweep, against the number of fixed-point
    # iterations of the attention inverse (Sec. 3.1 uses one), with recomputed and with remembered expert sets
    rel = lambda u, v: float(((u - v).double().norm() / v.double().norm()).item())
    recon = {}
    for remember in (False, True):
        for n in (1, 2, 3):
            step(iters=n, remember=remember)
            recon[f"iters={n},{'remembered' if remember else 'recomputed'}_routing"] = [rel(a, x1), rel(b, x2)]
    assert stk.status() == 0

    # end to end: streams and upstream gradients from pinned host memory, results back
    pin = lambda t: t.cpu().pin_memory()
    hx1, hx2, hd1, hd2 = pin(x1), pin(x2), pin(d1), pin(d2)
    ho = [torch.empty_like(hx1).pin_memory() for _ in range(4)]

    def host_step():
        a.copy_(hx1, non_blocking=True); b.copy_(hx2, non_blocking=True)
        g1.copy_(hd1, non_blocking=True); g2.copy_(hd2, non_blocking=True)
        stk.forward(a, b, None)
        stk.backward(a, b, g1, g2, ga, gm)
        for h, t in zip(ho, (a, b, g1, g2)):
            h.copy_(t, non_blocking=True)
        torch.cuda.synchronize()
    host_step()
    barrier()
    n_e2e = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        host_step()
    dt = max_over_ranks([time.perf_counter() - t0], world)[0] / n_e2e
    if rank != 0:
        return finish()

    cpu_rec = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import revffn_block_oracle as orc
        n_seq, S = 1, min(acfg.seq_len, 128)
        cut = lambda t: t.cpu().numpy().reshape(acfg.batch, acfg.seq_len, -1)[:n_seq, :S].reshape(n_seq * S, -1)
        pa = {n: t.float().cpu().numpy() for n, t in wa[0].items()}
        pm = {n: t.float().cpu().numpy() for n, t in wm[0].items()}
        cfg_o = dict(seq_len=S, n_heads=acfg.n_heads, n_kv_heads=acfg.n_kv_heads, top_k=mcfg.top_k, eps=mcfg.norm_eps,
                     theta=acfg.rope_theta)
        t0 = time.perf_counter()
        Y1, Y2, _ = orc.forward(pa, pm, cut(x1), cut(x2), cfg_o)
        orc.backward(pa, pm, Y1, Y2, cut(d1), cut(d2), cfg_o, n_iter=1)
        cdt = time.perf_counter() - t0
        cpu_rec = {"value": n_seq * S / cdt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                   "sample": f"one block (of {L}), forward + reversible backward over the first {S} positions of "
                             f"{n_seq} sequence, full weights, fp64 numpy, {cdt:.1f} s"}
    print(json.dumps({
        "metric": "RevFFN block stack fwd+reversible bwd tokens/s", "value": world * acfg.tokens / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{L} whole RevFFN blocks (attention branch Eq. 1 + MoE branch Eq. 2) of the "
                               f"Qwen1.5-MoE-A2.7B shape, {acfg.batch} x {acfg.seq_len} tokens per GPU; step = forward "
                               f"through all layers + reversible back-propagation (inverse pass with one fixed-point "
                               f"iteration, gradients at the rebuilt inputs, no cached activations); weights drawn "
                               f"on the device", "l2": "per-layer working set exceeds the 126 MB L2", "blocks": L,
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "ms_per_block": ms / L, "passes_ms": split, "gpu_launches": int(launches), "clocks": clocks,
        "memory": {"weights_bytes": w_bytes, "activation_bytes": act_bytes, "workspace_bytes": stk.bwd_bytes,
                   "peak_device_bytes": int(torch.cuda.max_memory_allocated()),
                   "note": "activation bytes = peak allocation above weights, input copies and the shared gradient "
                           "buffers while the stack ran: one workspace, two streams, two stream gradients, whatever "
                           "the number of layers"},
        "reconstruction_rel_l2_[x1,x2]": recon, "cpu_baseline": cpu_rec,
        "roofline": None,
        "e2e": {"value": world * acfg.tokens / dt, "unit": "tokens/s", "h2d_bytes_per_step": 4 * hx1.numel() * 4,
                "d2h_bytes_per_step": 4 * hx1.numel() * 4, "ms_per_step": dt * 1e3}}))
    finish()


def attn_flops(cfg):
    """Algorithmic flops per launch of the attention branch's matrix products, by profiler slot name.
    Causal attention needs half of the score and value products; the whole rectangle is counted
    where the kernel computes it, so 'useful' is stated beside it."""
    T, d, h, hd = cfg.tokens, cfg.d_model, cfg.h, cfg.head_dim
    dkv = cfg.n_kv_heads * hd
    S, rows = cfg.seq_len, cfg.batch * cfg.n_heads * cfg.seq_len
    core = 2 * rows * S * hd            # one full (rows x S x hd) product
    return {"gemm_p_up": 2 * T * h * d, "gemm_qkv": 2 * T * d * (d + 2 * dkv) / 3, "gemm_scores": core, "gemm_pv": core,
            "gemm_w_o": 2 * T * d * d, "gemm_p_down_couple": 2 * T * d * h, "gemm_dp": core, "gemm_dk_dv": core,
            "gemm_dq": core, "gemm_dn": 2 * (2 * T) * d * h,
            # scopes that cover several launches: average per scope
            "attn_wgrad": 2 * T * (h * d + 2 * d * d + 2 * dkv * d + 2 * d * h) / 6,
            "attn_dgrad": 2 * T * (d * h + 2 * d * d + 2 * dkv * d) / 4,
            # fused attention core, the causal half only: forward 2 products; gradient pass 7 (dK/dV 4, dQ 3)
            "flash_attention": core,
            "attn_bwd/flash_attention": (core + 3.5 * core) / 2}


def run_attn(args, cfg):
    """The attention coupling branch (Eq. 1) at cfg's shape: step = forward + inverse (one fixed-point
    iteration, Sec. 3.1) + backward by recomputation.  Prints one JSON line (rank 0)."""
    import torch
    import paper_2512_20920_b200 as rv
    from workloads.generate import make_attn_streams, make_attn_weights

    rank, world, local, barrier = dist_setup()
    w_host = make_attn_weights(cfg, args.seed)
    f32 = ("norm_gamma", "b_q", "b_k", "b_v")
    wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
    w_dev = {n: torch.from_numpy(v).cuda().to(torch.float32 if n in f32 else wdt).contiguous() for n, v in w_host.items()}
    s_host = make_attn_streams(cfg, replica_seed(args.seed, rank))
    br = rv.AttnBranch(batch=cfg.batch, seq_len=cfg.seq_len, d_model=cfg.d_model, n_heads=cfg.n_heads,
                       n_kv_heads=cfg.n_kv_heads, weight_dtype=rv.BF16 if cfg.weight_dtype == "bf16" else rv.F32,
                       weights=w_dev, norm_eps=cfg.norm_eps, rope_theta=cfg.rope_theta)
    x1, x2, dy1 = (torch.from_numpy(s_host[n]).cuda() for n in ("x1", "x2", "dy1"))
    y1, x1r, dx1, dx2 = torch.empty_like(x1), torch.empty_like(x1), torch.empty_like(x1), torch.zeros_like(x2)
    grads = {n: torch.empty(v.shape, dtype=torch.float32, device="cuda") for n, v in w_dev.items()}

    def step():
        br.forward(x1, x2, y1)
        br.inverse(y1, x2, x1r, n_iter=1)
        # the gradient pass takes keys and values from the inverse pass before it (same x2), as a block's
        # reversible back-propagation does
        br.backward(x1r, x2, dy1, dx2, dx1=dx1, grads=grads, reuse_kv=True)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    assert br.status() == 0

    def timed(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = rv.revffn_prof_launches()
    barrier()
    if sampler:
        sampler.start()
    ms_total = timed(step, args.steps)
    clocks = sampler.stop() if sampler else None
    launches = rv.revffn_prof_launches() - launches0
    assert br.status() == 0
    rv.revffn_prof_enable(True)
    barrier()
    sampler2 = ClockSampler(local) if rank == 0 else None
    if sampler2:
        sampler2.start()
    ms_prof_total = timed(step, args.steps)
    clocks_prof = sampler2.stop() if sampler2 else None
    if clocks_prof and not clocks_prof.get("sm_mhz"):
        clocks_prof = None
    prof = rv.revffn_prof_collect()
    rv.revffn_prof_enable(False)
    ms_total = max_over_ranks([ms_total], world)[0]
    ms_step = ms_total / args.steps

    # reconstruction error of the fixed-point inverse against the number of iterations (Sec. 3.1)
    recon = {}
    br.forward(x1, x2, y1)
    for n in (1, 2, 3, 4):
        xh = br.inverse(y1, x2, torch.empty_like(x1), n_iter=n)
        recon[str(n)] = float(((xh - x1).double().norm() / x1.double().norm()).item())
    recon["0"] = float(((y1 - x1).double().norm() / x1.double().norm()).item())

    # end to end: host-resident streams in, results out, copies inside the timed region
    pin = lambda a: torch.from_numpy(a).pin_memory()
    hx1, hx2, hdy1 = pin(s_host["x1"]), pin(s_host["x2"]), pin(s_host["dy1"])
    hy1, hx1r, hdx1 = (torch.empty_like(hx1).pin_memory() for _ in range(3))

    def host_step():
        x1.copy_(hx1, non_blocking=True); x2.copy_(hx2, non_blocking=True); dy1.copy_(hdy1, non_blocking=True)
        step()
        hy1.copy_(y1, non_blocking=True); hx1r.copy_(x1r, non_blocking=True); hdx1.copy_(dx1, non_blocking=True)
        torch.cuda.synchronize()
    host_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        host_step()
    dt = max_over_ranks([time.perf_counter() - t0], world)[0]
    if rank != 0:
        return finish()

    peaks, peak_kind = load_peaks()
    peak_t = peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"]
    flops = attn_flops(cfg)
    kernels = sorted(((ms, cnt, name, name.split("/")[1]) for name, (ms, cnt) in prof.items()), reverse=True)
    passes = {}
    for ms, cnt, name, kn in kernels:
        passes[name.split("/")[0]] = passes.get(name.split("/")[0], 0.0) + ms / args.steps
    fl = lambda name, kn: flops.get(name, flops.get(kn))
    top = [{"kernel": name, "ms_per_step": ms / args.steps, "launches_per_step": cnt / args.steps,
            "tflops": (fl(name, kn) * cnt / (ms * 1e-3) / 1e12) if fl(name, kn) and ms > 0 else None}
           for ms, cnt, name, kn in kernels]
    dom = next((k for k in kernels if fl(k[2], k[3])), None)
    roofline = None
    if dom:
        ms, cnt, name, kn = dom
        achieved = fl(name, kn) / (ms / cnt * 1e-3) / 1e12
        roofline = {"bound": "tensor", "kernel": name, "achieved": achieved, "peak": peak_t, "unit": "TFLOP/s",
                    "frac": achieved / peak_t, "peak_source": f"{peak_kind} (sustained bf16 cuBLAS figure)",
                    "traffic": None, "launch_ms": ms / cnt}
    cpu_rec = None
    if world == 1 and not args.no_cpu_baseline:
        from dataclasses import replace
        from oracle import revffn_attn_oracle as orc
        n_seq, S = 1, min(cfg.seq_len, 256)
        sub = {k: v.reshape(cfg.batch, cfg.seq_len, -1)[:n_seq, :S].reshape(n_seq * S, -1) for k, v in s_host.items()}
        kw = dict(S=S, n_heads=cfg.n_heads, n_kv_heads=cfg.n_kv_heads, eps=cfg.norm_eps, theta=cfg.rope_theta)
        t0 = time.perf_counter()
        Y = orc.forward(w_host, sub["x1"], sub["x2"], **kw)
        orc.inverse(w_host, Y, sub["x2"], n_iter=1, **kw)
        orc.backward(w_host, sub["x1"], sub["x2"], sub["dy1"], **kw)
        cdt = time.perf_counter() - t0
        cpu_rec = {"value": n_seq * S / cdt, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                   "sample": f"fwd+inverse+bwd over the first {S} positions of {n_seq} sequence, full weights, "
                             f"fp64 numpy, {cdt:.1f} s"}
    out = {
        "metric": "RevFFN attention branch fwd+inverse+bwd tokens/s", "value": job_tokens_per_s(world, cfg.tokens, args.steps, ms_total),
        "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: attention coupling branch of one Qwen1.5-MoE-A2.7B-shaped block, "
                               f"{cfg.batch} sequences x {cfg.seq_len} positions per GPU, d={cfg.d_model}, "
                               f"{cfg.n_heads} heads ({cfg.n_kv_heads} key/value heads) of {cfg.head_dim}; step = forward + "
                               f"inverse (one fixed-point iteration) + backward by recomputation (keys and values shared with the inverse pass), all weight gradients in fp32",
                   "l2": "per-step working set (score matrices alone 1 GB) exceeds the 126 MB L2",
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "passes_ms": passes, "kernels": top, "roofline": roofline, "cpu_baseline": cpu_rec,
        "reconstruction_rel_l2_by_iterations": recon,
        "e2e": {"value": job_tokens_per_s(world, cfg.tokens, args.steps, dt * 1e3), "unit": "tokens/s",
                "h2d_bytes_per_step": 3 * hx1.numel() * 4, "d2h_bytes_per_step": 3 * hx1.numel() * 4,
                "ms_per_step": 1e3 * dt / args.steps},
        "gpu_launches": int(launches), "clocks": clocks, "peak_device_bytes": int(torch.cuda.max_memory_allocated()),
        "workspace_bytes": {"fwd": br.fwd_bytes, "bwd": br.bwd_bytes},
        "profiled_ms_per_step": ms_prof_total / args.steps,
    }
    print(json.dumps(out))
    finish()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C1")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-sample-tokens", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--steps-only", action="store_true",
                    help="single-block runs: warm-up and the timed steps only (no per-kernel pass, no unshared variant, no "
                         "end-to-end or CPU leg) -- the short command the profiler captures are taken from")
    ap.add_argument("--blocks", type=int, default=0, help="C3: number of layers (default: the configuration's 24)")
    ap.add_argument("--no-drift", action="store_true", help="C3: skip the per-layer drift pass")
    ap.add_argument("--seq-len", type=int, default=0, help="A1: sequence length at the same token count (default 2048)")
    ap.add_argument("--gating", default="renorm", choices=["renorm", "softmax_all"],
                    help="single-block runs: gate weights renormalised over the top-k (default, the benchmark's "
                         "definition) or taken from the softmax over all experts")
    args = ap.parse_args()
    from workloads import CONFIGS
    from workloads.generate import ATTN_CONFIGS
    if args.config in ("B1", "B3") and args.impl == "ours":
        return run_block_stack(args, ATTN_CONFIGS["A1"], CONFIGS["C1"], 24 if args.config == "B3" else 1)
    if args.config in ATTN_CONFIGS and args.impl == "ours":
        acfg = ATTN_CONFIGS[args.config]
        if args.seq_len:        # same number of tokens in fewer, longer (or more, shorter) sequences
            from dataclasses import replace
            acfg = replace(acfg, seq_len=args.seq_len, batch=max(1, acfg.tokens // args.seq_len),
                           name=f"{acfg.name}@seq{args.seq_len}")
        return run_attn(args, acfg)
    if args.impl == "reference" and args.config not in CONFIGS:
        args.config = "C1"          # the reference arm times the oracle of the headline path only
    if args.config == "C4":
        if args.impl == "reference":
            args.config = "C1"
        else:
            return run_sweep(args)
    cfg = CONFIGS[args.config]
    if args.cpu_sample_tokens is None:
        args.cpu_sample_tokens = min(cfg.tokens, 128 if args.impl == "ours" else 64)
    if args.impl == "reference":
        run_reference(args, cfg)
    elif cfg.n_blocks > 1:
        run_stack(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
