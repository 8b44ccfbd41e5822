"""Seeded synthetic tensors for the benchmark configurations.

Shapes follow the block the paper wraps (Sec. 3.1, Eq. 2; Sec. 3.2 adapters):
two d/2-wide fp32 streams, adapters d/2 -> d and d -> d/2, and a
Qwen1.5-MoE-A2.7B-shaped sparse MoE (router, routed SwiGLU experts, gated
shared SwiGLU expert) in between.  Values: streams ~ N(0,1), weights
~ N(0,0.02), norm scale 1 + N(0,0.02).  Nothing here evaluates the block.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Iterable, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class BlockConfig:
    name: str
    tokens: int          # T = batch * seq, flattened
    d_model: int         # d; each stream is h = d/2 wide
    n_experts: int       # E
    top_k: int           # k
    d_expert: int        # I, routed SwiGLU intermediate
    d_shared: int        # I_s, shared SwiGLU intermediate (0 = no shared expert)
    weight_dtype: str    # "f32" | "bf16"
    norm_eps: float = 1e-6
    zipf_s: Optional[float] = None   # skewed routing: load ~ rank^-s
    n_blocks: int = 1

    @property
    def h(self) -> int:
        return self.d_model // 2

    def with_tokens(self, tokens: int) -> "BlockConfig":
        return replace(self, tokens=tokens, name=f"{self.name}@{tokens}")


_QWEN = dict(d_model=2048, n_experts=60, top_k=4, d_expert=1408, d_shared=5632,
             weight_dtype="bf16")

CONFIGS: Dict[str, BlockConfig] = {
    # tiny fp32 block, no shared expert
    "C0": BlockConfig("C0", tokens=64, d_model=128, n_experts=8, top_k=2,
                      d_expert=256, d_shared=0, weight_dtype="f32"),
    # Qwen1.5-MoE-A2.7B-shaped block, batch 4 x seq 2048
    "C1": BlockConfig("C1", tokens=8192, **_QWEN),
    # same block, Zipf(1.2) expert load, two experts guaranteed empty
    "C2": BlockConfig("C2", tokens=16384, zipf_s=1.2, **_QWEN),
    # 24-block reversible stack of C1
    "C3": BlockConfig("C3", tokens=8192, n_blocks=24, **_QWEN),
}
for _t in (512, 2048, 8192, 32768, 65536):
    CONFIGS[f"C4-{_t}"] = BlockConfig(f"C4-{_t}", tokens=_t, **_QWEN)

# tensor ids: fixed so that every tensor has its own random stream
_TENSOR_IDS = {
    "norm_gamma": 1, "w_up": 2, "w_down": 3, "w_router": 4, "b_router": 5,
    "w_gate": 6, "w_upx": 7, "w_downx": 8, "ws_gate": 9, "ws_up": 10,
    "ws_down": 11, "ws_sgate": 12, "y1": 20, "x2": 21, "dy2": 22, "perm": 30,
}


def _gen(seed: int, block: int, name: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1_000_003 + int(block) * 7919) * 64 + _TENSOR_IDS[name])
    return g


def to_bf16_values(x: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16 value (ties to even), kept as fp32."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def _normal(shape, std, mean, seed, block, name, bf16):
    t = torch.randn(shape, generator=_gen(seed, block, name), dtype=torch.float32)
    t = t * std + mean
    if bf16:
        t = t.to(torch.bfloat16).to(torch.float32)
    return t.numpy()


# Bias scale for the skewed-routing configuration: b[pi(j)] = ALPHA * ln p_j with
# p_j ~ j^-s.  ALPHA was chosen once, offline, so that the routed load of the
# upper ranks falls with slope about -s in log-log at the C2 shape (a selection of
# k experts without replacement caps any share at 1/k, so rank 1 saturates).
ZIPF_ALPHA = 0.325
ZIPF_EMPTY_BIAS = -30.0
ZIPF_N_EMPTY = 2


def zipf_router_bias(n_experts: int, s: float, seed: int, block: int = 0,
                     alpha: float = ZIPF_ALPHA) -> np.ndarray:
    """Router bias that skews expert load towards rank^-s; the last
    ZIPF_N_EMPTY ranks get a bias so low that they are never selected."""
    ranks = np.arange(1, n_experts + 1, dtype=np.float64)
    p = ranks ** (-float(s))
    p /= p.sum()
    perm = torch.randperm(n_experts, generator=_gen(seed, block, "perm")).numpy()
    b = np.empty(n_experts, dtype=np.float32)
    b[perm] = (alpha * np.log(p)).astype(np.float32)
    b[perm[n_experts - ZIPF_N_EMPTY:]] = ZIPF_EMPTY_BIAS
    return b


def weight_shapes(cfg: BlockConfig) -> Dict[str, tuple]:
    """Name -> shape of every weight of one block, row-major [out, in]."""
    d, h, E, I, Is = cfg.d_model, cfg.h, cfg.n_experts, cfg.d_expert, cfg.d_shared
    shapes = {
        "norm_gamma": (h,), "w_up": (d, h), "w_down": (h, d), "w_router": (E, d),
        "w_gate": (E, I, d), "w_upx": (E, I, d), "w_downx": (E, d, I),
    }
    if cfg.zipf_s is not None:
        shapes["b_router"] = (E,)
    if Is > 0:
        shapes.update(ws_gate=(Is, d), ws_up=(Is, d), ws_down=(d, Is), ws_sgate=(d,))
    return shapes


def make_weights(cfg: BlockConfig, seed: int = 0, block: int = 0,
                 only: Optional[Iterable[str]] = None) -> Dict[str, np.ndarray]:
    """Weights of one block as fp32 arrays, row-major [out, in].  With
    weight_dtype == "bf16" every matrix value is exactly representable in bf16.
    `only` restricts the draw to the named tensors (each has its own stream)."""
    bf = cfg.weight_dtype == "bf16"
    w = {}
    for name, shape in weight_shapes(cfg).items():
        if only is not None and name not in only:
            continue
        if name == "norm_gamma":
            w[name] = _normal(shape, 0.02, 1.0, seed, block, name, False)
        elif name == "b_router":
            w[name] = zipf_router_bias(cfg.n_experts, cfg.zipf_s, seed, block)
        else:
            w[name] = _normal(shape, 0.02, 0.0, seed, block, name, bf)
    return w


def make_streams(cfg: BlockConfig, seed: int = 0) -> Dict[str, np.ndarray]:
    """Input streams Y1, X2 and the upstream gradient dY2, each [T, h] fp32 ~ N(0,1)."""
    T, h = cfg.tokens, cfg.h
    return {name: _normal((T, h), 1.0, 0.0, seed, 0, name, False)
            for name in ("y1", "x2", "dy2")}


def make_weights_device(cfg: BlockConfig, seed: int = 0, block: int = 0, device: str = "cuda") -> Dict[str, torch.Tensor]:
    """Weights of one block drawn on `device` in their final dtypes (bf16 or fp32 matrices,
    fp32 norm scale and router bias): same shapes and distributions as `make_weights`, its own
    seeded streams.  For stacks whose weights are too large to draw on the host in reasonable
    time; a CPU reference reads the same bytes back with `.cpu()`."""
    wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
    out = {}
    for name, shape in weight_shapes(cfg).items():
        g = torch.Generator(device=device)
        g.manual_seed((int(seed) * 1_000_003 + int(block) * 7919) * 64 + _TENSOR_IDS[name] + (1 << 40))
        if name == "b_router":
            out[name] = torch.from_numpy(zipf_router_bias(cfg.n_experts, cfg.zipf_s, seed, block)).to(device)
            continue
        n = int(np.prod(shape))
        # drawn in slices to bound the fp32 scratch of a large tensor
        t = torch.empty(n, dtype=torch.float32 if name == "norm_gamma" else wdt, device=device)
        step = 1 << 27
        for i in range(0, n, step):
            m = min(step, n - i)
            v = torch.randn(m, generator=g, device=device, dtype=torch.float32) * 0.02
            if name == "norm_gamma":
                v = v + 1.0
            t[i:i + m] = v.to(t.dtype)
        out[name] = t.view(shape)
    return out


# --------------------------------------------------------------------------- #
# Attention coupling branch (Sec. 3.1 Eq. 1): shapes of the same base model's attention layer
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class AttnConfig:
    name: str
    batch: int           # sequences
    seq_len: int         # positions per sequence; T = batch * seq_len tokens
    d_model: int
    n_heads: int
    n_kv_heads: int
    weight_dtype: str    # "f32" | "bf16"
    norm_eps: float = 1e-6
    rope_theta: float = 1e6

    @property
    def h(self) -> int:
        return self.d_model // 2

    @property
    def tokens(self) -> int:
        return self.batch * self.seq_len

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads


ATTN_CONFIGS: Dict[str, AttnConfig] = {
    # tiny fp32 branch with grouped key/value heads and a ragged sequence length
    "A0": AttnConfig("A0", batch=2, seq_len=40, d_model=64, n_heads=4, n_kv_heads=2, weight_dtype="f32"),
    # Qwen1.5-MoE-A2.7B-shaped attention layer, batch 4 x seq 2048 (the token batch of C1)
    "A1": AttnConfig("A1", batch=4, seq_len=2048, d_model=2048, n_heads=16, n_kv_heads=16, weight_dtype="bf16"),
}

_ATTN_IDS = {"norm_gamma": 41, "w_up": 42, "w_down": 43, "w_q": 44, "w_k": 45, "w_v": 46, "w_o": 47,
             "b_q": 48, "b_k": 49, "b_v": 50, "x1": 55, "x2": 56, "dy1": 57, "dx2": 58}
_TENSOR_IDS.update({"attn." + k: v for k, v in _ATTN_IDS.items()})


def attn_weight_shapes(cfg: AttnConfig) -> Dict[str, tuple]:
    d, h, dkv = cfg.d_model, cfg.h, cfg.n_kv_heads * cfg.head_dim
    return {"norm_gamma": (h,), "w_up": (d, h), "w_down": (h, d), "w_q": (d, d), "w_k": (dkv, d), "w_v": (dkv, d),
            "w_o": (d, d), "b_q": (d,), "b_k": (dkv,), "b_v": (dkv,)}


def make_attn_weights(cfg: AttnConfig, seed: int = 0, std: float = 0.02, bias_std: float = 0.02) -> Dict[str, np.ndarray]:
    """Weights of one attention branch as fp32 arrays, row-major [out, in]; with weight_dtype "bf16"
    every matrix value is exactly representable in bf16 (norm scale and biases stay fp32)."""
    bf = cfg.weight_dtype == "bf16"
    w = {}
    for name, shape in attn_weight_shapes(cfg).items():
        if name == "norm_gamma":
            w[name] = _normal(shape, 0.02, 1.0, seed, 0, "attn." + name, False)
        elif name.startswith("b_"):
            w[name] = _normal(shape, bias_std, 0.0, seed, 0, "attn." + name, False)
        else:
            w[name] = _normal(shape, std, 0.0, seed, 0, "attn." + name, bf)
    return w


def make_attn_streams(cfg: AttnConfig, seed: int = 0) -> Dict[str, np.ndarray]:
    """Input streams X1, X2, the upstream gradient dY1 and a starting value for dX2, each [T, h] fp32 ~ N(0,1)."""
    return {name: _normal((cfg.tokens, cfg.h), 1.0, 0.0, seed, 0, "attn." + name, False)
            for name in ("x1", "x2", "dy1", "dx2")}


def make_attn_weights_device(cfg: AttnConfig, seed: int = 0, block: int = 0, device: str = "cuda") -> Dict[str, torch.Tensor]:
    """Attention-branch weights of one block drawn on `device` in their final dtypes: same shapes and
    distributions as `make_attn_weights`, its own seeded streams (for stacks too large to draw on the host)."""
    wdt = torch.bfloat16 if cfg.weight_dtype == "bf16" else torch.float32
    out = {}
    for name, shape in attn_weight_shapes(cfg).items():
        g = torch.Generator(device=device)
        g.manual_seed((int(seed) * 1_000_003 + int(block) * 7919) * 64 + _ATTN_IDS[name] + (1 << 41))
        v = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * 0.02
        if name == "norm_gamma":
            v = v + 1.0
        out[name] = v.to(torch.float32 if name == "norm_gamma" or name.startswith("b_") else wdt).contiguous()
    return out
